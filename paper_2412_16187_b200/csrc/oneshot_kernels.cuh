// he_prefill_oneshot: prompt compression by the averaged-Hamming ranking of Appendix C (the paper's global-ranking
// simulation; NOT the procedure of Section 3). Per unit and prompt token i, with the group's G query heads summed as
// in Eq. 5:
//   S_i = sum_{j > i} sum_g popc(h(k_i) xor h(q_{j,g})),   average_i = S_i / (N - 1 - i)   (0 for the last token);
// the min(N, C) tokens with the lowest average stay (protected windows first, equal averages by token index).
//
// The double sum is linear in per-bit counts, so no N x N pass is needed: with later_i[k] = number of (j > i, g) whose
// query code has bit k set,  S_i = sum_k ( bit_k(h(k_i)) ? (N-1-i) G - later_i[k] : later_i[k] ).  A lane owns bit k
// (and k + 32), keeps later[k] in a register while its warp walks a chunk of tokens backwards, and one redux.sync
// per token adds the lanes' terms. O(N (G + b)) integer work per unit, all of it exact.
//
// Selection is exact as well: averages are compared through the key floor(S 2^32 / n), which orders any two
// fractions with denominators below 2^15 like the fractions themselves (they differ by at least 2^-30), the token
// index is appended, and a radix select (8 bits per pass) finds the min(N, C)-th smallest key.
#pragma once
#include "common.cuh"

namespace he {

struct OneshotArgs {
  he_config cfg;
  he_cache ca;
  const uint32_t* kcodes;  // [units, Nmax, Wd]
  const uint32_t* qcodes;  // [units, Nmax, G, Wd]
  const int32_t* prompt_len;
  long long Nmax;
  int32_t* sums;             // scratch [units, Nmax]: S_i
  unsigned long long* keys;  // scratch [units, Nmax]: selection keys
  long long* sums_out;       // optional [units, Nmax]: S_i for the caller
};

constexpr int kOneshotThreads = 512;
constexpr int kOneshotWarps = kOneshotThreads / 32;
constexpr int kOneshotSub = 32;  // tokens staged per warp at a time
constexpr unsigned long long kOneshotRanked = 1ull << 57;  // set in the keys of tokens outside the protected windows

// Squared L2 norm of every prompt key in the precision that decides the L2 ranking: fp32, channels in ascending order,
// one fused multiply-add per channel starting from 0. One thread per row (the chain is sequential by definition);
// the float's bit pattern goes to the `sums` scratch, which the ranking kernel reads as its sort key.
struct NormArgs {
  he_config cfg;
  const void* k;
  long long s0, s1, s2;  // element strides (batch, head, token)
  const int32_t* prompt_len;
  long long Nmax;
  int32_t* norm_bits;  // scratch [units, Nmax]
  float* norms_out;    // optional [units, Nmax]
};

__global__ void __launch_bounds__(kOneshotThreads) key_norms_kernel(const NormArgs a) {
  const long long unit = blockIdx.y;
  const int s = (int)(unit / a.cfg.n_kv_heads), h = (int)(unit % a.cfg.n_kv_heads);
  const int i = blockIdx.x * kOneshotThreads + threadIdx.x;
  if (i >= min(a.prompt_len[s], (int)a.Nmax)) return;
  const int d = a.cfg.head_dim, es = esize_of(a.cfg.dtype);
  const char* row = static_cast<const char*>(a.k) + (s * a.s0 + h * a.s1 + (long long)i * a.s2) * es;
  float acc = 0.f;
  for (int c0 = 0; c0 < d * es / 16; ++c0) {  // 16 bytes at a time: 8 bf16 or 4 fp32 channels
    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(row) + c0);
    const uint32_t wv[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (a.cfg.dtype == HE_DTYPE_BF16) {
        const float lo = __uint_as_float(wv[k] << 16), hi = __uint_as_float(wv[k] & 0xFFFF0000u);
        acc = fmaf(lo, lo, acc);
        acc = fmaf(hi, hi, acc);
      } else {
        const float x = __uint_as_float(wv[k]);
        acc = fmaf(x, x, acc);
      }
    }
  }
  a.norm_bits[unit * a.Nmax + i] = __float_as_int(acc);
  if (a.norms_out != nullptr) a.norms_out[unit * a.Nmax + i] = acc;
}

// POLICY 0: averaged Hamming distance (Appendix C). POLICY 1: squared key norm, ascending (the comparison policy the
// paper names); `sums` then holds the norms' bit patterns written by key_norms_kernel, qcodes is not read.
template <int WORDS, int POLICY>
__global__ void __launch_bounds__(kOneshotThreads) oneshot_rank_kernel(const OneshotArgs a) {
  __shared__ int chunk_cnt[kOneshotWarps][32 * WORDS];
  __shared__ uint32_t qbuf[POLICY == 0 ? kOneshotWarps : 1][kOneshotSub * kMaxGroup * WORDS];  // staged query codes, per warp
  __shared__ uint32_t kbuf[POLICY == 0 ? kOneshotWarps : 1][kOneshotSub * WORDS];              // staged key codes
  __shared__ unsigned int hist[256];
  __shared__ unsigned long long s_prefix;
  __shared__ int s_want;
  __shared__ int s_scan[kOneshotThreads];
  const he_config& cfg = a.cfg;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long unit = blockIdx.x;
  const int s = (int)(unit / cfg.n_kv_heads);
  const int G = cfg.group_size, GW = G * WORDS;
  const long long Cmax = cfg.max_budget;
  const int C = clamp_budget(a.ca.budget[s], (int)Cmax);
  const int N = clamp_len(a.prompt_len[s], a.Nmax, C);
  const int keep = N < C ? N : C;
  const uint32_t* kc_u = a.kcodes + unit * a.Nmax * WORDS;
  const uint32_t* qc_u = a.qcodes + unit * a.Nmax * GW;
  int32_t* S = a.sums + unit * a.Nmax;
  unsigned long long* keys = a.keys + unit * a.Nmax;

  // ---- (1) S_i. Tokens are split into one contiguous chunk per warp; a lane counts the ones of its bits. Codes go
  // through a per-warp shared-memory buffer, kOneshotSub tokens at a time, so that global loads are coalesced and
  // the per-token loop reads broadcast words instead of waiting on a dependent global load.
  if (POLICY == 0) {
    uint32_t* qb = qbuf[warp];
    uint32_t* kb = kbuf[warp];
    const int chunk = (N + kOneshotWarps - 1) / kOneshotWarps;
    const int lo = min(N, warp * chunk), hi = min(N, lo + chunk);
    int cnt[WORDS];
#pragma unroll
    for (int w = 0; w < WORDS; ++w) cnt[w] = 0;
    for (int j0 = lo; j0 < hi; j0 += kOneshotSub) {  // ones per bit over this warp's chunk
      const int nt = min(kOneshotSub, hi - j0);
      for (int x = lane; x < nt * GW; x += 32) qb[x] = __ldg(qc_u + (long long)j0 * GW + x);
      __syncwarp();
#pragma unroll 4
      for (int x = 0; x < nt * G; ++x) {
#pragma unroll
        for (int w = 0; w < WORDS; ++w) cnt[w] += (qb[x * WORDS + w] >> lane) & 1u;
      }
      __syncwarp();
    }
#pragma unroll
    for (int w = 0; w < WORDS; ++w) chunk_cnt[warp][w * 32 + lane] = cnt[w];
    __syncthreads();
#pragma unroll
    for (int w = 0; w < WORDS; ++w) {  // ones per bit over all later chunks
      cnt[w] = 0;
      for (int x = warp + 1; x < kOneshotWarps; ++x) cnt[w] += chunk_cnt[x][w * 32 + lane];
    }
    for (int j1 = hi; j1 > lo; j1 -= kOneshotSub) {  // sub-chunks from the back; cnt = ones per bit over the tokens j > i
      const int j0 = max(lo, j1 - kOneshotSub), nt = j1 - j0;
      for (int x = lane; x < nt * GW; x += 32) qb[x] = __ldg(qc_u + (long long)j0 * GW + x);
      for (int x = lane; x < nt * WORDS; x += 32) kb[x] = __ldg(kc_u + (long long)j0 * WORDS + x);
      __syncwarp();
#pragma unroll 2
      for (int t = nt - 1; t >= 0; --t) {
        const int i = j0 + t;
        const int m = (N - 1 - i) * G;
        int term = 0;
#pragma unroll
        for (int w = 0; w < WORDS; ++w) {
          const uint32_t hbit = (kb[t * WORDS + w] >> lane) & 1u;
          term += hbit ? m - cnt[w] : cnt[w];
        }
        const int Si = __reduce_add_sync(0xFFFFFFFFu, term);
        if (lane == (t & 31)) {  // spread the stores over the lanes
          S[i] = Si;
          if (a.sums_out != nullptr) a.sums_out[unit * a.Nmax + i] = Si;
        }
        for (int g = 0; g < G; ++g) {
#pragma unroll
          for (int w = 0; w < WORDS; ++w) cnt[w] += (qb[(t * G + g) * WORDS + w] >> lane) & 1u;
        }
      }
      __syncwarp();
    }
    __syncthreads();
  }

  // ---- (2) keys: protected tokens sort first in token order, the others by average, then index
  for (int i = tid; i < N; i += kOneshotThreads) {
    const bool prot = i < cfg.n_sink || i >= N - cfg.n_recent;
    const int n = N - 1 - i;
    unsigned long long key = (unsigned long long)i;
    if (!prot) {
      unsigned long long q;
      if (POLICY == 0) q = n > 0 ? ((unsigned long long)(uint32_t)S[i] << 32) / (unsigned long long)n : 0ull;
      else q = (unsigned long long)(uint32_t)S[i];  // bits of a non-negative float order like the float
      key = kOneshotRanked | (q << 15) | (unsigned long long)i;
    }
    keys[i] = key;
  }
  __syncthreads();

  // ---- (3) the keep-th smallest key by radix select, 8 bits per pass from the top (keys are distinct)
  unsigned long long thresh = ~0ull;
  if (keep < N) {
    if (tid == 0) {
      s_prefix = 0ull;
      s_want = keep;
    }
    for (int shift = 56; shift >= 0; shift -= 8) {
      if (tid < 256) hist[tid] = 0u;
      __syncthreads();
      const unsigned long long prefix = s_prefix;
      for (int i = tid; i < N; i += kOneshotThreads) {
        const unsigned long long key = keys[i];
        if (shift == 56 || (key >> (shift + 8)) == prefix) atomicAdd(&hist[(unsigned)(key >> shift) & 255u], 1u);
      }
      __syncthreads();
      if (tid == 0) {
        int want = s_want, bin = 0;
        while (bin < 255 && (int)hist[bin] < want) want -= (int)hist[bin++];
        s_want = want;
        s_prefix = (prefix << 8) | (unsigned long long)bin;
      }
      __syncthreads();
    }
    thresh = s_prefix;
  }

  // ---- (4) kept tokens in token order: slot = number of kept tokens before this one
  const int per = (N + kOneshotThreads - 1) / kOneshotThreads;
  const int b0 = min(N, tid * per), b1 = min(N, b0 + per);
  int mine = 0;
  for (int i = b0; i < b1; ++i) mine += keys[i] <= thresh ? 1 : 0;
  s_scan[tid] = mine;
  __syncthreads();
  if (tid == 0) {
    int run = 0;
    for (int t = 0; t < kOneshotThreads; ++t) {
      const int c = s_scan[t];
      s_scan[t] = run;
      run += c;
    }
  }
  __syncthreads();
  int slot = s_scan[tid];
  for (int i = b0; i < b1; ++i) {
    if (keys[i] <= thresh) {
      const long long dst = unit * Cmax + slot;
      uint32_t cw[WORDS];
#pragma unroll
      for (int w = 0; w < WORDS; ++w) cw[w] = kc_u[(long long)i * WORDS + w];
      store_slot_code<WORDS>(a.cfg, a.ca.codes, dst, cw);
      a.ca.pos[dst] = i;
      const int n = N - 1 - i;
      a.ca.scores[dst] = POLICY == 0 ? (n > 0 ? -((float)S[i] / (float)n) : 0.f) : -__int_as_float(S[i]);
      ++slot;
    }
  }
  for (int j = keep + tid; j < Cmax; j += kOneshotThreads) {  // everything beyond `fill` is reset
    uint32_t cw[WORDS];
#pragma unroll
    for (int w = 0; w < WORDS; ++w) cw[w] = 0u;
    store_slot_code<WORDS>(a.cfg, a.ca.codes, unit * Cmax + j, cw);
    a.ca.pos[unit * Cmax + j] = -1;
    a.ca.scores[unit * Cmax + j] = 0.f;
  }
  if (tid == 0) {
    a.ca.fill[unit] = keep;
    a.ca.next_pos[unit] = N;
  }
}

// he_decode_step_l2: one decoding step of the L2-norm comparison policy, one CTA per unit. scores[j] = -norm2 of the
// key in slot j (kept by he_prefill_oneshot_l2 and by this kernel), so the victim is the eligible slot with the lowest
// score, lowest slot on equal scores; if no slot is eligible, all are. The new key's norm is the same sequential fp32
// chain as in key_norms_kernel (thread 0), computed while the others scan.
struct StepL2Args {
  he_config cfg;
  he_cache ca;
  const void* k;  // [B, Hkv, d]
  const void* v;
  int32_t* victim_out;
  int32_t* evicted_pos_out;
};

constexpr int kStepL2Threads = 128;

__global__ void __launch_bounds__(kStepL2Threads) decode_step_l2_kernel(const StepL2Args a) {
  __shared__ unsigned long long wbest[2][kStepL2Threads / 32];
  __shared__ float s_norm;
  const he_config& cfg = a.cfg;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long unit = (long long)blockIdx.y * cfg.n_kv_heads + blockIdx.x;
  const int d = cfg.head_dim, es = esize_of(cfg.dtype), Wd = (cfg.hash_bits + 31) / 32;
  const long long Cmax = cfg.max_budget;
  const int C = clamp_budget(a.ca.budget[blockIdx.y], (int)Cmax);
  const int fill = min(a.ca.fill[unit], C), t = a.ca.next_pos[unit];
  if (C < 1) {  // a unit without a budget holds nothing: report it and leave the state alone
    if (tid == 0) {
      a.victim_out[unit] = -1;
      if (a.evicted_pos_out != nullptr) a.evicted_pos_out[unit] = -1;
    }
    return;
  }
  const char* kr = static_cast<const char*>(a.k) + unit * d * es;
  const char* vr = static_cast<const char*>(a.v) + unit * d * es;
  if (tid == 0) {
    float acc = 0.f;
    for (int c = 0; c < d; ++c) {
      const float x = cfg.dtype == HE_DTYPE_BF16 ? bf16_bits_to_f32(reinterpret_cast<const uint16_t*>(kr)[c])
                                                 : reinterpret_cast<const float*>(kr)[c];
      acc = fmaf(x, x, acc);
    }
    s_norm = acc;
  }
  int slot = fill;
  if (fill >= C) {
    // key = bits of norm2 (a non-negative float: ordered like its bits) above the inverted slot index
    unsigned long long best_all = 0ull, best_el = 0ull;
    const float* sc = a.ca.scores + unit * Cmax;
    const int32_t* pp = a.ca.pos + unit * Cmax;
    for (int j = tid; j < fill; j += kStepL2Threads) {
      const unsigned long long key =
          ((unsigned long long)__float_as_uint(-sc[j]) << 24) | (unsigned long long)(0xFFFFFF - j) | (1ull << 60);
      best_all = max(best_all, key);
      const int p = pp[j];
      if (p >= cfg.n_sink && p < t - cfg.n_recent) best_el = max(best_el, key);
    }
    for (int o = 16; o > 0; o >>= 1) {
      best_all = max(best_all, __shfl_xor_sync(0xFFFFFFFFu, best_all, o));
      best_el = max(best_el, __shfl_xor_sync(0xFFFFFFFFu, best_el, o));
    }
    if (lane == 0) wbest[0][warp] = best_all, wbest[1][warp] = best_el;
    __syncthreads();
    unsigned long long fa = 0ull, fe = 0ull;
    for (int w = 0; w < kStepL2Threads / 32; ++w) fa = max(fa, wbest[0][w]), fe = max(fe, wbest[1][w]);
    const unsigned long long fin = fe != 0ull ? fe : fa;
    slot = 0xFFFFFF - (int)(fin & 0xFFFFFFull);
  } else {
    __syncthreads();
  }
  if (!HE_IN_RANGE(slot, C)) return;
  const long long dst = unit * Cmax + slot;
  for (int i = tid; i < 2 * (d * es / 16); i += kStepL2Threads) {
    const int half = d * es / 16;
    const bool is_k = i < half;
    const uint4 row = __ldg(reinterpret_cast<const uint4*>(is_k ? kr : vr) + (is_k ? i : i - half));
    reinterpret_cast<uint4*>(static_cast<char*>(is_k ? a.ca.k_cache : a.ca.v_cache) + dst * d * es)[is_k ? i : i - half] = row;
  }
  if (tid == 0) {
    int ev = -1;
    if (fill >= C) ev = a.ca.pos[dst];
    a.ca.pos[dst] = t;
    a.ca.scores[dst] = -s_norm;
    if (const int cb = packed_code_bytes(a.cfg)) {
      for (int w = 0; w < cb; ++w) reinterpret_cast<uint8_t*>(a.ca.codes)[dst * cb + w] = 0;
    } else {
      for (int w = 0; w < Wd; ++w) a.ca.codes[dst * Wd + w] = 0u;
    }
    if (fill < C) a.ca.fill[unit] = fill + 1;
    a.ca.next_pos[unit] = t + 1;
    a.victim_out[unit] = slot;
    if (a.evicted_pos_out != nullptr) a.evicted_pos_out[unit] = ev;
  }
}

}  // namespace he
