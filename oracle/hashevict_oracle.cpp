// CPU oracle for the HashEvict eviction path. TEST INFRASTRUCTURE ONLY.
//
// Plain, slow, single-purpose C++: it is the procedure of Section 3 written out step by
// step so that it can be checked against the paper by eye. It shares no code with the CUDA
// library and is never called by it; only the tests, the smoke check and the benchmark's
// cpu_baseline / reference legs load it.
//
// What each function follows:
//   orc_hash            Eq. 2: h(x) = sgn(R x), sgn(p) = 1 if p >= 0 else 0; W = R^T is [d, b].
//   unit_step           Eq. 5 (F_score = -d_H(h(q), H)), Eq. 6 (e_t = argmin F_score) and
//                       Algorithm 1 lines 1-5 (evict slot e_t, insert k_t, v_t, h(k_t)).
//   orc_prefill*        "Prompt Encoding Stage": the first C tokens fill the cache, then
//                       Algorithm 1 runs for every later prompt token in order.
//   orc_step*           "Decoding Stage": Algorithm 1 continued, one call per generated token.
//
//   orc_attend          Eq. 1 on the compressed cache (Algorithm 1 line 6): softmax(q K^T / sqrt(d)) V per query head,
//                       over the valid slots of the head's KV unit, in fp64.
//
// Readings taken where the paper is silent (all restated in the design notes):
//   * q_t is compared with the table BEFORE k_t is inserted (Algorithm 1 line 1).
//   * arg-min ties go to the lowest slot index; the victim's slot is overwritten in place.
//   * grouped-query attention: the G query heads of a KV head add their Hamming distances.
//   * protected tokens (first n_sink positions, n_recent newest cached positions) are skipped
//     by the arg-min; if that leaves nothing, protection is ignored for that step.
//   * while the cache is not full the token is appended and no score is computed.
//   * a score is the integer -D stored as fp32; it is overwritten each step, never accumulated.
//
// Pins (tests/test_oracle_pins.py): Eq. 2 against a library matmul in fp64, scale invariance,
// h(-x) = ~h(x), sgn(0) = 1; Eq. 3 (E[d_H]/b = theta/pi) at known angles; brute force of the
// victim rule on tiny caches with unpacked bit arrays; the constant-budget and newest-resident
// invariants; codes == hash(K) for every slot; prefill == reset + N steps; the storage closed
// form of Section 4.7; orc_attend against a library softmax-attention in fp64, a single-slot cache, equal keys (mean
// of V), invariance to the slot order. Parity unpinned: none.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>

typedef struct orc_config {
  int32_t batch;       // sequences (layers may be folded in by the caller)
  int32_t n_kv_heads;  // KV heads per sequence
  int32_t group_size;  // G query heads per KV head
  int32_t head_dim;    // d
  int32_t hash_bits;   // b
  int32_t max_budget;  // Cmax: slot stride of the cache arrays
  int32_t n_sink;      // first n_sink prompt positions are never evicted
  int32_t n_recent;    // the n_recent newest cached positions are never evicted
  int32_t dtype;       // 0 = fp32, 1 = bf16 (for K, Q, V and the caches)
} orc_config;

typedef struct orc_cache {
  void* k_cache;          // [B, Hkv, Cmax, d]
  void* v_cache;          // [B, Hkv, Cmax, d]
  uint32_t* codes;        // [B, Hkv, Cmax, Wd]
  float* scores;          // [B, Hkv, Cmax]
  int32_t* pos;           // [B, Hkv, Cmax] token position held by the slot, -1 = empty
  const int32_t* budget;  // [B] C_s
  int32_t* fill;          // [B, Hkv] valid slots
  int32_t* next_pos;      // [B, Hkv] position t of the next token
} orc_cache;

static inline int words_of(int b) { return (b + 31) / 32; }
static inline int esize(int dtype) { return dtype ? 2 : 4; }

static inline double load_elem(const void* p, int64_t i, int dtype) {
  if (dtype == 0) return (double)((const float*)p)[i];
  uint32_t u = (uint32_t)((const uint16_t*)p)[i] << 16;  // bf16 is the top half of an fp32
  float f;
  std::memcpy(&f, &u, 4);
  return (double)f;
}

// Eq. 2 for one vector x[d]: code bit i = [ sum_c x_c * W[c, i] >= 0 ], bit i in word i/32, LSB first.
// fragile bit i is set when |p_i| < 1e-5 * ||x|| * ||W[:, i]|| (the only bits an fp32 device
// projection is allowed to get wrong).
static void hash_one(const void* x, int dtype, int d, const float* W, int b, uint32_t* code, uint32_t* fragile,
                     double* proj) {
  const int Wd = words_of(b);
  for (int w = 0; w < Wd; ++w) {
    code[w] = 0;
    if (fragile) fragile[w] = 0;
  }
  double xnorm2 = 0.0;
  for (int c = 0; c < d; ++c) {
    const double xc = load_elem(x, c, dtype);
    xnorm2 += xc * xc;
  }
  for (int i = 0; i < b; ++i) {
    double p = 0.0;
    for (int c = 0; c < d; ++c) p += load_elem(x, c, dtype) * (double)W[(int64_t)c * b + i];
    if (p >= 0.0) code[i / 32] |= (1u << (i % 32));
    if (fragile) {
      double wnorm2 = 0.0;
      for (int c = 0; c < d; ++c) wnorm2 += (double)W[(int64_t)c * b + i] * (double)W[(int64_t)c * b + i];
      if (std::fabs(p) < 1e-5 * std::sqrt(xnorm2) * std::sqrt(wnorm2)) fragile[i / 32] |= (1u << (i % 32));
    }
    if (proj) proj[i] = p;
  }
}

// Hash `rows` vectors. codes_out / fragile_out are [rows, Wd]; proj_out (nullable) is [rows, b] fp64.
extern "C" void orc_hash(const void* x, int64_t rows, int64_t row_stride_elems, int32_t d, int32_t dtype, const float* W, int32_t b,
              uint32_t* codes_out, uint32_t* fragile_out, double* proj_out) {
  const int Wd = words_of(b);
  for (int64_t r = 0; r < rows; ++r) {
    const char* xr = (const char*)x + r * row_stride_elems * esize(dtype);
    hash_one(xr, dtype, d, W, b, codes_out + r * Wd, fragile_out ? fragile_out + r * Wd : nullptr,
             proj_out ? proj_out + r * b : nullptr);
  }
}

static inline int hamming(const uint32_t* a, const uint32_t* bb, int Wd) {
  int dist = 0;
  for (int w = 0; w < Wd; ++w) {
    uint32_t x = a[w] ^ bb[w];
    while (x) {  // count differing bits one at a time
      dist += (int)(x & 1u);
      x >>= 1;
    }
  }
  return dist;
}

// One application of Algorithm 1 (lines 1-5) to one (sequence, KV head) unit, given the codes.
//   qc: [G, Wd] query codes of the group, kc: [Wd] code of the new key, k / v: the new rows [d].
static void unit_step(const orc_config* cfg, const orc_cache* ca, int64_t unit, int32_t C, const uint32_t* qc,
                      const uint32_t* kc, const void* k, const void* v, int32_t* victim_out, int32_t* evicted_pos_out) {
  const int Wd = words_of(cfg->hash_bits), d = cfg->head_dim, G = cfg->group_size, es = esize(cfg->dtype);
  const int64_t Cmax = cfg->max_budget;
  uint32_t* codes = ca->codes + unit * Cmax * Wd;
  float* scores = ca->scores + unit * Cmax;
  int32_t* pos = ca->pos + unit * Cmax;
  char* kc_rows = (char*)ca->k_cache + unit * Cmax * d * es;
  char* vc_rows = (char*)ca->v_cache + unit * Cmax * d * es;
  const int32_t fill = ca->fill[unit];
  const int32_t t = ca->next_pos[unit];

  int32_t slot, evicted = -1;
  if (fill < C) {
    slot = fill;  // cache not full yet: append, nothing is scored
    scores[slot] = 0.0f;
  } else {
    // Eq. 5: score_j = -d_H(h(q), H_j), summed over the G query heads of the group.
    std::vector<int> D(fill);
    for (int32_t j = 0; j < fill; ++j) {
      int dist = 0;
      for (int g = 0; g < G; ++g) dist += hamming(codes + (int64_t)j * Wd, qc + g * Wd, Wd);
      D[j] = dist;
      scores[j] = -(float)dist;
    }
    // Eq. 6: lowest score = largest distance; first such eligible slot wins.
    slot = -1;
    int best = -1;
    for (int32_t j = 0; j < fill; ++j) {
      const bool eligible = pos[j] >= cfg->n_sink && pos[j] < t - cfg->n_recent;
      if (eligible && D[j] > best) {
        best = D[j];
        slot = j;
      }
    }
    if (slot < 0) {  // everything protected: ignore protection for this step
      for (int32_t j = 0; j < fill; ++j)
        if (D[j] > best) {
          best = D[j];
          slot = j;
        }
    }
    evicted = pos[slot];
  }
  // Algorithm 1 lines 2-5: the victim's K, V and code are replaced by the new token's.
  std::memcpy(kc_rows + (int64_t)slot * d * es, k, (size_t)d * es);
  std::memcpy(vc_rows + (int64_t)slot * d * es, v, (size_t)d * es);
  for (int w = 0; w < Wd; ++w) codes[(int64_t)slot * Wd + w] = kc[w];
  pos[slot] = t;
  ca->next_pos[unit] = t + 1;
  ca->fill[unit] = fill < C ? fill + 1 : fill;
  if (victim_out) victim_out[unit] = slot;
  if (evicted_pos_out) evicted_pos_out[unit] = evicted;
}

template <class F>
static void for_units(int64_t n, int threads, F f) {
  if (threads <= 1) {
    for (int64_t u = 0; u < n; ++u) f(u);
    return;
  }
  std::vector<std::thread> pool;
  for (int th = 0; th < threads; ++th)
    pool.emplace_back([=]() {
      for (int64_t u = th; u < n; u += threads) f(u);
    });
  for (auto& t : pool) t.join();
}

// fill = 0, next_pos = 0, pos = -1, codes = 0, scores = 0; K / V untouched.
extern "C" void orc_reset(const orc_config* cfg, orc_cache* ca) {
  const int64_t units = (int64_t)cfg->batch * cfg->n_kv_heads, Cmax = cfg->max_budget;
  const int Wd = words_of(cfg->hash_bits);
  for (int64_t u = 0; u < units; ++u) {
    ca->fill[u] = 0;
    ca->next_pos[u] = 0;
    for (int64_t j = 0; j < Cmax; ++j) {
      ca->pos[u * Cmax + j] = -1;
      ca->scores[u * Cmax + j] = 0.0f;
      for (int w = 0; w < Wd; ++w) ca->codes[(u * Cmax + j) * Wd + w] = 0;
    }
  }
}

// One decode step on given codes: qcodes [B, Hkv*G, Wd], kcodes [B, Hkv, Wd], k / v [B, Hkv, d].
extern "C" void orc_step_codes(const orc_config* cfg, orc_cache* ca, const uint32_t* qcodes, const uint32_t* kcodes, const void* k,
                    const void* v, int32_t* victim_out, int32_t* evicted_pos_out, int32_t threads) {
  const int Wd = words_of(cfg->hash_bits), d = cfg->head_dim, G = cfg->group_size, es = esize(cfg->dtype);
  const int64_t units = (int64_t)cfg->batch * cfg->n_kv_heads;
  for_units(units, threads, [=](int64_t u) {
    const int32_t C = ca->budget[u / cfg->n_kv_heads];
    unit_step(cfg, ca, u, C, qcodes + u * G * Wd, kcodes + u * Wd, (const char*)k + u * d * es, (const char*)v + u * d * es,
              victim_out, evicted_pos_out);
  });
}

// One decode step from the embeddings: hashes q [B, Hkv*G, d] and k [B, Hkv, d] with Eq. 2, then as above.
// qcodes_out [B, Hkv*G, Wd] and kcodes_out [B, Hkv, Wd] are nullable.
extern "C" void orc_step(const orc_config* cfg, orc_cache* ca, const float* W, const void* q, const void* k, const void* v,
              int32_t* victim_out, int32_t* evicted_pos_out, uint32_t* qcodes_out, uint32_t* kcodes_out, int32_t threads) {
  const int Wd = words_of(cfg->hash_bits), d = cfg->head_dim, G = cfg->group_size;
  const int64_t units = (int64_t)cfg->batch * cfg->n_kv_heads;
  std::vector<uint32_t> qc((size_t)units * G * Wd), kc((size_t)units * Wd);
  orc_hash(q, units * G, d, d, cfg->dtype, W, cfg->hash_bits, qc.data(), nullptr, nullptr);
  orc_hash(k, units, d, d, cfg->dtype, W, cfg->hash_bits, kc.data(), nullptr, nullptr);
  if (qcodes_out) std::memcpy(qcodes_out, qc.data(), qc.size() * 4);
  if (kcodes_out) std::memcpy(kcodes_out, kc.data(), kc.size() * 4);
  orc_step_codes(cfg, ca, qc.data(), kc.data(), k, v, victim_out, evicted_pos_out, threads);
}

// Prompt encoding on given codes. kcodes [B, Hkv, Nmax, Wd]; qcodes [B, Hkv, Nmax, G, Wd] (entries of
// tokens that are appended are never read). k, v: strided [B, Hkv, N, d]; strides in elements
// (batch, head, token). prompt_len [B]. The cache is reset first.
extern "C" void orc_prefill_codes(const orc_config* cfg, orc_cache* ca, const uint32_t* kcodes, const uint32_t* qcodes, const void* k,
                       const void* v, const int64_t* kv_strides, const int32_t* prompt_len, int32_t max_prompt_len,
                       int32_t threads) {
  const int Wd = words_of(cfg->hash_bits), G = cfg->group_size, es = esize(cfg->dtype);
  const int64_t units = (int64_t)cfg->batch * cfg->n_kv_heads, Nmax = max_prompt_len;
  orc_reset(cfg, ca);
  for_units(units, threads, [=](int64_t u) {
    const int64_t s = u / cfg->n_kv_heads, h = u % cfg->n_kv_heads;
    const int32_t C = ca->budget[s], N = prompt_len[s];
    for (int32_t t = 0; t < N; ++t) {
      const int64_t off = (s * kv_strides[0] + h * kv_strides[1] + (int64_t)t * kv_strides[2]) * es;
      unit_step(cfg, ca, u, C, qcodes + ((u * Nmax + t) * G) * Wd, kcodes + (u * Nmax + t) * Wd, (const char*)k + off,
                (const char*)v + off, nullptr, nullptr);
    }
  });
}

// Prompt encoding from the embeddings: q strided [B, Hkv*G, N, d], k / v strided [B, Hkv, N, d].
// kcodes_out [B, Hkv, Nmax, Wd] and qcodes_out [B, Hkv, Nmax, G, Wd] are nullable; when given they
// receive the Eq. 2 codes of every prompt token (queries of appended tokens included).
extern "C" void orc_prefill(const orc_config* cfg, orc_cache* ca, const float* W, const void* q, const void* k, const void* v,
                 const int64_t* q_strides, const int64_t* kv_strides, const int32_t* prompt_len, int32_t max_prompt_len,
                 uint32_t* kcodes_out, uint32_t* qcodes_out, int32_t threads) {
  const int Wd = words_of(cfg->hash_bits), G = cfg->group_size, d = cfg->head_dim, es = esize(cfg->dtype);
  const int64_t units = (int64_t)cfg->batch * cfg->n_kv_heads, Nmax = max_prompt_len;
  std::vector<uint32_t> kc((size_t)units * Nmax * Wd, 0u), qc((size_t)units * Nmax * G * Wd, 0u);
  uint32_t* kcp = kc.data();
  uint32_t* qcp = qc.data();
  for_units(units, threads, [=](int64_t u) {
    const int64_t s = u / cfg->n_kv_heads, h = u % cfg->n_kv_heads;
    const int32_t N = prompt_len[s];
    for (int32_t t = 0; t < N; ++t) {
      const int64_t koff = (s * kv_strides[0] + h * kv_strides[1] + (int64_t)t * kv_strides[2]) * es;
      hash_one((const char*)k + koff, cfg->dtype, d, W, cfg->hash_bits, kcp + (u * Nmax + t) * Wd, nullptr, nullptr);
      for (int g = 0; g < G; ++g) {
        const int64_t qoff = (s * q_strides[0] + (h * G + g) * q_strides[1] + (int64_t)t * q_strides[2]) * es;
        hash_one((const char*)q + qoff, cfg->dtype, d, W, cfg->hash_bits, qcp + ((u * Nmax + t) * G + g) * Wd, nullptr,
                 nullptr);
      }
    }
  });
  if (kcodes_out) std::memcpy(kcodes_out, kc.data(), kc.size() * 4);
  if (qcodes_out) std::memcpy(qcodes_out, qc.data(), qc.size() * 4);
  orc_prefill_codes(cfg, ca, kc.data(), qc.data(), k, v, kv_strides, prompt_len, max_prompt_len, threads);
}


// One-shot ranking by averaged Hamming distance (Appendix C: "the average Hamming distance between the key code of
// token i and the query codes of all tokens j > i", tokens sorted from lowest to highest average). This is the
// paper's global-ranking simulation, NOT the procedure of Section 3; here it is written out as a prompt-compression
// variant: the C best-ranked tokens stay. Per unit, with the group's G query heads summed as in Eq. 5:
//   S_i = sum_{j > i} sum_g popc(h(k_i) xor h(q_{j,g})),   n_i = N - 1 - i,   average_i = S_i / n_i  (0 when n_i = 0).
// Order: tokens inside the protected windows (i < n_sink or i >= N - n_recent) first, in token order; then by
// average, compared exactly as fractions (S_a n_b < S_b n_a); equal averages by token index. The first min(N, C)
// tokens of that order are kept and stored in token order: slot s holds the s-th kept token (its K, V, code and
// position; score = -(float)S / (float)n, 0 when n = 0). kcodes [B, Hkv, Nmax, Wd]; qcodes [B, Hkv, Nmax, G, Wd];
// sums_out [B, Hkv, Nmax] int64 (nullable) receives S_i. The cache is reset first.
extern "C" void orc_oneshot_codes(const orc_config* cfg, orc_cache* ca, const uint32_t* kcodes, const uint32_t* qcodes,
                                  const void* k, const void* v, const int64_t* kv_strides, const int32_t* prompt_len,
                                  int32_t max_prompt_len, int64_t* sums_out, int32_t threads) {
  const int Wd = words_of(cfg->hash_bits), G = cfg->group_size, d = cfg->head_dim, es = esize(cfg->dtype);
  const int64_t units = (int64_t)cfg->batch * cfg->n_kv_heads, Nmax = max_prompt_len, Cmax = cfg->max_budget;
  orc_reset(cfg, ca);
  for_units(units, threads, [=](int64_t u) {
    const int64_t s = u / cfg->n_kv_heads, h = u % cfg->n_kv_heads;
    const int32_t C = ca->budget[s], N = prompt_len[s];
    std::vector<int64_t> S(N, 0);
    for (int32_t i = 0; i < N; ++i) {
      const uint32_t* hi = kcodes + (u * Nmax + i) * Wd;
      int64_t acc = 0;
      for (int32_t j = i + 1; j < N; ++j)
        for (int g = 0; g < G; ++g) {
          const uint32_t* hq = qcodes + ((u * Nmax + j) * G + g) * Wd;
          for (int w = 0; w < Wd; ++w) acc += __builtin_popcount(hi[w] ^ hq[w]);
        }
      S[i] = acc;
      if (sums_out) sums_out[u * Nmax + i] = acc;
    }
    std::vector<int32_t> order(N);
    for (int32_t i = 0; i < N; ++i) order[i] = i;
    auto prot = [&](int32_t i) { return i < cfg->n_sink || i >= N - cfg->n_recent; };
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
      const bool pa = prot(a), pb = prot(b);
      if (pa != pb) return pa;
      if (pa) return a < b;
      const int64_t na = N - 1 - a > 0 ? N - 1 - a : 1, nb = N - 1 - b > 0 ? N - 1 - b : 1;  // S = 0 when n = 0
      const int64_t lhs = S[a] * nb, rhs = S[b] * na;
      if (lhs != rhs) return lhs < rhs;
      return a < b;
    });
    const int32_t keep = N < C ? N : C;
    std::vector<int32_t> kept(order.begin(), order.begin() + keep);
    std::sort(kept.begin(), kept.end());
    for (int32_t sl = 0; sl < keep; ++sl) {
      const int32_t t = kept[sl];
      const int64_t slot = u * Cmax + sl;
      const int64_t off = (s * kv_strides[0] + h * kv_strides[1] + (int64_t)t * kv_strides[2]) * es;
      std::memcpy((char*)ca->k_cache + slot * d * es, (const char*)k + off, (size_t)d * es);
      std::memcpy((char*)ca->v_cache + slot * d * es, (const char*)v + off, (size_t)d * es);
      for (int w = 0; w < Wd; ++w) ca->codes[slot * Wd + w] = kcodes[(u * Nmax + t) * Wd + w];
      ca->pos[slot] = t;
      const int64_t n = N - 1 - t;
      ca->scores[slot] = n > 0 ? -((float)S[t] / (float)n) : 0.0f;
    }
    ca->fill[u] = keep;
    ca->next_pos[u] = N;
  });
}

// Squared L2 norm of a key row in the precision that decides the L2 ranking: fp32, channels in ascending order, one
// fused multiply-add per channel starting from 0 (the inputs are widened exactly).
static inline float norm2_f32(const void* x, int dtype, int d) {
  float acc = 0.0f;
  for (int c = 0; c < d; ++c) {
    const float xc = (float)load_elem(x, c, dtype);
    acc = std::fmaf(xc, xc, acc);
  }
  return acc;
}

// The comparison policy the paper names (Section 1 / Section 4 setup: "dropping tokens based on the high L2 norms of
// their key embeddings"; Appendix B calls its ranking "a low-to-high ordering of all L2 key norms"), as a one-shot
// prompt-compression variant under the same boundary: tokens inside the protected windows first (token order), then
// by squared key norm ascending, equal norms by token index; the first min(N, C) stay, stored in token order. Slot s
// holds the s-th kept token: K, V, its Eq. 2 code (so that the cache remains a valid state for Algorithm 1), position,
// score = -norm2. norms_out [B, Hkv, Nmax] (nullable) receives norm2 of every prompt key. The cache is reset first.
extern "C" void orc_oneshot_l2(const orc_config* cfg, orc_cache* ca, const uint32_t* kcodes, const void* k, const void* v,
                               const int64_t* kv_strides, const int32_t* prompt_len, int32_t max_prompt_len,
                               float* norms_out, int32_t threads) {
  const int Wd = words_of(cfg->hash_bits), d = cfg->head_dim, es = esize(cfg->dtype);
  const int64_t units = (int64_t)cfg->batch * cfg->n_kv_heads, Nmax = max_prompt_len, Cmax = cfg->max_budget;
  orc_reset(cfg, ca);
  for_units(units, threads, [=](int64_t u) {
    const int64_t s = u / cfg->n_kv_heads, h = u % cfg->n_kv_heads;
    const int32_t C = ca->budget[s], N = prompt_len[s];
    std::vector<float> nrm(N);
    for (int32_t i = 0; i < N; ++i) {
      const int64_t off = (s * kv_strides[0] + h * kv_strides[1] + (int64_t)i * kv_strides[2]) * es;
      nrm[i] = norm2_f32((const char*)k + off, cfg->dtype, d);
      if (norms_out) norms_out[u * Nmax + i] = nrm[i];
    }
    std::vector<int32_t> order(N);
    for (int32_t i = 0; i < N; ++i) order[i] = i;
    auto prot = [&](int32_t i) { return i < cfg->n_sink || i >= N - cfg->n_recent; };
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
      const bool pa = prot(a), pb = prot(b);
      if (pa != pb) return pa;
      if (pa) return a < b;
      if (nrm[a] != nrm[b]) return nrm[a] < nrm[b];
      return a < b;
    });
    const int32_t keep = N < C ? N : C;
    std::vector<int32_t> kept(order.begin(), order.begin() + keep);
    std::sort(kept.begin(), kept.end());
    for (int32_t sl = 0; sl < keep; ++sl) {
      const int32_t t = kept[sl];
      const int64_t slot = u * Cmax + sl;
      const int64_t off = (s * kv_strides[0] + h * kv_strides[1] + (int64_t)t * kv_strides[2]) * es;
      std::memcpy((char*)ca->k_cache + slot * d * es, (const char*)k + off, (size_t)d * es);
      std::memcpy((char*)ca->v_cache + slot * d * es, (const char*)v + off, (size_t)d * es);
      for (int w = 0; w < Wd; ++w) ca->codes[slot * Wd + w] = kcodes[(u * Nmax + t) * Wd + w];
      ca->pos[slot] = t;
      ca->scores[slot] = -nrm[t];
    }
    ca->fill[u] = keep;
    ca->next_pos[u] = N;
  });
}

// One decoding step of the L2-norm comparison policy under the same boundary as Algorithm 1: the new token always
// enters; while the cache is full the resident token with the HIGHEST squared key norm leaves (lowest slot on equal
// norms; protected windows as in Algorithm 1, ignored for a step in which no slot is eligible). It relies on
// scores[j] = -norm2 of the key in slot j, which orc_oneshot_l2 and this function maintain; the code of the slot is
// set to zero (this policy has no use for it). k / v: [B, Hkv, d].
extern "C" void orc_step_l2(const orc_config* cfg, orc_cache* ca, const void* k, const void* v, int32_t* victim_out,
                            int32_t* evicted_pos_out, int32_t threads) {
  const int Wd = words_of(cfg->hash_bits), d = cfg->head_dim, es = esize(cfg->dtype);
  const int64_t units = (int64_t)cfg->batch * cfg->n_kv_heads, Cmax = cfg->max_budget;
  for_units(units, threads, [=](int64_t u) {
    const int32_t C = ca->budget[u / cfg->n_kv_heads];
    float* scores = ca->scores + u * Cmax;
    int32_t* pos = ca->pos + u * Cmax;
    const int32_t fill = ca->fill[u], t = ca->next_pos[u];
    const char* kr = (const char*)k + u * d * es;
    const char* vr = (const char*)v + u * d * es;
    int32_t slot = fill, evicted = -1;
    if (fill >= C) {
      slot = -1;
      for (int pass = 0; pass < 2 && slot < 0; ++pass) {  // second pass: nothing was eligible, so everything is
        float worst = 0.0f;
        for (int32_t j = 0; j < fill; ++j) {
          const bool eligible = pass == 1 || (pos[j] >= cfg->n_sink && pos[j] < t - cfg->n_recent);
          if (eligible && (slot < 0 || scores[j] < worst)) {
            worst = scores[j];
            slot = j;
          }
        }
      }
      evicted = pos[slot];
    }
    std::memcpy((char*)ca->k_cache + (u * Cmax + slot) * d * es, kr, (size_t)d * es);
    std::memcpy((char*)ca->v_cache + (u * Cmax + slot) * d * es, vr, (size_t)d * es);
    for (int w = 0; w < Wd; ++w) ca->codes[(u * Cmax + slot) * Wd + w] = 0u;
    scores[slot] = -norm2_f32(kr, cfg->dtype, d);
    pos[slot] = t;
    ca->next_pos[u] = t + 1;
    ca->fill[u] = fill < C ? fill + 1 : fill;
    if (victim_out) victim_out[u] = slot;
    if (evicted_pos_out) evicted_pos_out[u] = evicted;
  });
}

// Attention loss of a compressed cache (Section 4.6 / Appendix B: "the sum of the attention probabilities for the
// evicted tokens. Or equivalently, 1 - the sum of the attention probabilities for the tokens in the compressed
// cache"). For every unit and each of its G query heads, with a = softmax_p(q_g . k_p / sqrt(d)) over ALL n = next_pos
// tokens seen so far (k_full strided [B, Hkv, n, d]):  loss = 1 - sum_{valid slots j} a[pos_j].  out [B, Hkv*G] fp64.
// A unit that has seen no token gives 0.
extern "C" void orc_attention_loss(const orc_config* cfg, const orc_cache* ca, const void* q, const void* k_full,
                                   const int64_t* kv_strides, double* out) {
  const int d = cfg->head_dim, G = cfg->group_size, es = esize(cfg->dtype);
  const int64_t units = (int64_t)cfg->batch * cfg->n_kv_heads, Cmax = cfg->max_budget;
  for (int64_t u = 0; u < units; ++u) {
    const int64_t s = u / cfg->n_kv_heads, h = u % cfg->n_kv_heads;
    const int n = ca->next_pos[u], fill = ca->fill[u];
    for (int g = 0; g < G; ++g) {
      const char* qg = (const char*)q + (u * G + g) * d * es;
      if (n == 0) {
        out[u * G + g] = 0.0;
        continue;
      }
      std::vector<double> a(n);
      double mx = -INFINITY;
      for (int p = 0; p < n; ++p) {
        const char* kp = (const char*)k_full + (s * kv_strides[0] + h * kv_strides[1] + (int64_t)p * kv_strides[2]) * es;
        double dot = 0.0;
        for (int c = 0; c < d; ++c) dot += load_elem(qg, c, cfg->dtype) * load_elem(kp, c, cfg->dtype);
        a[p] = dot / std::sqrt((double)d);
        if (a[p] > mx) mx = a[p];
      }
      double den = 0.0;
      for (int p = 0; p < n; ++p) {
        a[p] = std::exp(a[p] - mx);
        den += a[p];
      }
      double keptsum = 0.0;
      for (int j = 0; j < fill; ++j) keptsum += a[ca->pos[u * Cmax + j]] / den;
      out[u * G + g] = 1.0 - keptsum;
    }
  }
}

// Eq. 1 over the compressed cache (Algorithm 1 line 6): for every unit and each of its G query heads,
//   out[g] = sum_j softmax_j( q_g . K_j / sqrt(d) ) V_j   over the valid slots j < fill.
// q: [B, Hkv*G, d] in the cache dtype; out: [B, Hkv*G, d] fp64. A unit with no valid slot gives zeros.
extern "C" void orc_attend(const orc_config* cfg, const orc_cache* ca, const void* q, double* out) {
  const int d = cfg->head_dim, G = cfg->group_size, es = esize(cfg->dtype);
  const int64_t units = (int64_t)cfg->batch * cfg->n_kv_heads, Cmax = cfg->max_budget;
  for (int64_t u = 0; u < units; ++u) {
    const int fill = ca->fill[u];
    const char* K = (const char*)ca->k_cache + u * Cmax * d * es;
    const char* V = (const char*)ca->v_cache + u * Cmax * d * es;
    for (int g = 0; g < G; ++g) {
      const char* qg = (const char*)q + (u * G + g) * d * es;
      double* o = out + (u * G + g) * d;
      for (int c = 0; c < d; ++c) o[c] = 0.0;
      if (fill == 0) continue;
      std::vector<double> sc(fill);
      double mx = -INFINITY;
      for (int j = 0; j < fill; ++j) {
        double dot = 0.0;
        for (int c = 0; c < d; ++c) dot += load_elem(qg, c, cfg->dtype) * load_elem(K, (int64_t)j * d + c, cfg->dtype);
        sc[j] = dot / std::sqrt((double)d);
        if (sc[j] > mx) mx = sc[j];
      }
      double den = 0.0;
      for (int j = 0; j < fill; ++j) {
        sc[j] = std::exp(sc[j] - mx);
        den += sc[j];
      }
      for (int j = 0; j < fill; ++j)
        for (int c = 0; c < d; ++c) o[c] += (sc[j] / den) * load_elem(V, (int64_t)j * d + c, cfg->dtype);
    }
  }
}
