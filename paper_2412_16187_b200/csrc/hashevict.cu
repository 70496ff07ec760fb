// HashEvict eviction hot path for B200 (sm_100a): kernels and the C ABI declared in include/hashevict.h.
//
// Kernels in this file
//   hash_rows_kernel       Eq. 2 on many rows: x tile and W staged in shared memory, one lane per hash bit,
//                          sign bits packed with warp ballots.
//   decode_step_kernel     Algorithm 1 lines 1-5 for one unit per CTA: code words are pulled into registers with
//                          16-byte loads while the new q/k rows are hashed, then XOR+popcount, packed arg-max
//                          (redux.sync + one block barrier), in-place overwrite of the victim slot.
//   prefill_replay_kernel  the prompt-encoding loop of Section 3 for one unit per CTA, code table resident in
//                          shared memory, one block barrier per token.
//   prefill_gather_kernel  copies the surviving K/V rows into their slots.
//   reset_kernel           empties the cache.
//
// One projection order is used by every path (bulk hash, decode, prefill) so that they produce the same bits:
// channels are cut into chunks of 32; a chunk's partial sum is an fmaf chain in ascending channel order starting
// from 0; the partial sums are added in ascending chunk order; the bit is (sum >= 0).
#include <cuda_runtime.h>

#include <cstdarg>
#include <cstdio>
#include <cstring>

#include "hashevict.h"

namespace {

thread_local char g_err[512] = "";

int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

#define HE_CUDA_CHECK(expr)                                                                         \
  do {                                                                                              \
    cudaError_t e_ = (expr);                                                                        \
    if (e_ != cudaSuccess) return fail(HE_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e_)); \
  } while (0)

constexpr int kChunk = 32;        // channels per partial sum of the projection
constexpr int kMaxDim = 256;      // largest head_dim
constexpr int kMaxGroup = 8;      // largest group size
constexpr int kKeyIdxBits = 20;   // arg-max key = (D + 1) << 20 | (0xFFFFF - slot)
constexpr uint32_t kKeyIdxMask = (1u << kKeyIdxBits) - 1u;

__host__ __device__ inline int words_of(int b) { return (b + 31) >> 5; }
__host__ __device__ inline int esize_of(int dtype) { return dtype == HE_DTYPE_BF16 ? 2 : 4; }

__device__ __forceinline__ float bf16_bits_to_f32(uint32_t h) { return __uint_as_float(h << 16); }

__device__ __forceinline__ uint32_t word_mask(int b, int w) {
  const int n = b - 32 * w;
  return n >= 32 ? 0xFFFFFFFFu : (n <= 0 ? 0u : ((1u << n) - 1u));
}

// Copies 16 bytes (8 bf16 or 4 fp32) of a row into fp32 shared memory.
__device__ __forceinline__ void stage_chunk(float* dst, const void* src_row, int chunk, int dtype) {
  const uint4 raw = __ldg(reinterpret_cast<const uint4*>(src_row) + chunk);
  if (dtype == HE_DTYPE_BF16) {
    float* o = dst + chunk * 8;
    const uint32_t wds[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      o[2 * i] = bf16_bits_to_f32(wds[i] & 0xFFFFu);
      o[2 * i + 1] = bf16_bits_to_f32(wds[i] >> 16);
    }
  } else {
    float* o = dst + chunk * 4;
    o[0] = __uint_as_float(raw.x);
    o[1] = __uint_as_float(raw.y);
    o[2] = __uint_as_float(raw.z);
    o[3] = __uint_as_float(raw.w);
  }
}

// ------------------------------------------------------------------------------------------------ bulk hash

constexpr int kHashThreads = 256;
constexpr int kHashRows = 128;  // rows per CTA
constexpr int kHashRpw = 16;    // rows per warp

struct HashJob {
  const void* x;
  const float* W;
  uint32_t* out;
  int mode;  // 0: flat rows; 1: prompt keys; 2: prompt queries
  int dtype, d, b;
  long long rows, row_stride;  // mode 0
  long long s0, s1, s2;        // modes 1, 2: element strides (batch, head, token)
  int heads, G, Hkv;           // heads = heads per sequence of this tensor
  long long Nmax;
  const int32_t* prompt_len;
  const int32_t* budget;
};

template <int WORDS>
__global__ void __launch_bounds__(kHashThreads) hash_rows_kernel(const HashJob job) {
  extern __shared__ __align__(16) float hsm[];
  constexpr int BP = 32 * WORDS;
  const int d = job.d, b = job.b, es = esize_of(job.dtype);
  float* Ws = hsm;            // [d][BP]
  float* xs = hsm + d * BP;   // [kHashRows][d]

  // which rows does this CTA hash, and where do the codes go
  const char* base;
  long long stride, r_begin, r_end, out_base, out_stride;
  if (job.mode == 0) {
    base = static_cast<const char*>(job.x);
    stride = job.row_stride;
    r_begin = 0;
    r_end = job.rows;
    out_base = 0;
    out_stride = WORDS;
  } else {
    const int seg = blockIdx.y;
    const int s = seg / job.heads, hh = seg % job.heads;
    const long long N = job.prompt_len[s];
    const long long C = job.budget[s];
    base = static_cast<const char*>(job.x) + (s * job.s0 + hh * job.s1) * es;
    stride = job.s2;
    r_end = N;
    if (job.mode == 1) {
      r_begin = 0;
      out_base = ((long long)s * job.Hkv + hh) * job.Nmax * WORDS;
      out_stride = WORDS;
    } else {
      r_begin = C < N ? C : N;  // queries of appended tokens are never read
      const long long unit = (long long)s * job.Hkv + hh / job.G;
      out_base = (unit * job.Nmax * job.G + hh % job.G) * WORDS;
      out_stride = (long long)job.G * WORDS;
    }
  }
  const long long row0 = r_begin + (long long)blockIdx.x * kHashRows;
  if (row0 >= r_end) return;
  const int nrows = (int)((r_end - row0) < kHashRows ? (r_end - row0) : kHashRows);

  for (int idx = threadIdx.x; idx < d * BP; idx += kHashThreads) {
    const int c = idx / BP, i = idx % BP;
    Ws[idx] = i < b ? __ldg(job.W + (long long)c * b + i) : 0.f;
  }
  const int cpr = d * es / 16;  // 16-byte chunks per row
  for (int idx = threadIdx.x; idx < kHashRows * cpr; idx += kHashThreads) {
    const int r = idx / cpr, ch = idx % cpr;
    if (r < nrows) {
      stage_chunk(xs + r * d, base + (row0 + r) * stride * es, ch, job.dtype);
    } else {
      float* o = xs + r * d + ch * (16 / es);
      for (int i = 0; i < 16 / es; ++i) o[i] = 0.f;
    }
  }
  __syncthreads();

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float* xw = xs + warp * kHashRpw * d;
  float tot[kHashRpw][WORDS];
#pragma unroll
  for (int r = 0; r < kHashRpw; ++r)
#pragma unroll
    for (int w = 0; w < WORDS; ++w) tot[r][w] = 0.f;

  for (int c0 = 0; c0 < d; c0 += kChunk) {
    float acc[kHashRpw][WORDS];
#pragma unroll
    for (int r = 0; r < kHashRpw; ++r)
#pragma unroll
      for (int w = 0; w < WORDS; ++w) acc[r][w] = 0.f;
    const int cend = (d - c0) < kChunk ? (d - c0) : kChunk;
    for (int cc = 0; cc < cend; cc += 4) {
      float wv[4][WORDS];
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int w = 0; w < WORDS; ++w) wv[k][w] = Ws[(c0 + cc + k) * BP + lane + 32 * w];
#pragma unroll
      for (int r = 0; r < kHashRpw; ++r) {
        const float4 xv = *reinterpret_cast<const float4*>(xw + r * d + c0 + cc);
#pragma unroll
        for (int w = 0; w < WORDS; ++w) {
          acc[r][w] = fmaf(xv.x, wv[0][w], acc[r][w]);
          acc[r][w] = fmaf(xv.y, wv[1][w], acc[r][w]);
          acc[r][w] = fmaf(xv.z, wv[2][w], acc[r][w]);
          acc[r][w] = fmaf(xv.w, wv[3][w], acc[r][w]);
        }
      }
    }
#pragma unroll
    for (int r = 0; r < kHashRpw; ++r)
#pragma unroll
      for (int w = 0; w < WORDS; ++w) tot[r][w] += acc[r][w];
  }

  uint32_t mine[WORDS];
#pragma unroll
  for (int w = 0; w < WORDS; ++w) mine[w] = 0u;
#pragma unroll
  for (int r = 0; r < kHashRpw; ++r)
#pragma unroll
    for (int w = 0; w < WORDS; ++w) {
      const uint32_t word = __ballot_sync(0xFFFFFFFFu, tot[r][w] >= 0.f) & word_mask(b, w);
      if (lane == r) mine[w] = word;
    }
  const int r = warp * kHashRpw + lane;
  if (lane < kHashRpw && r < nrows) {
    uint32_t* o = job.out + out_base + (row0 + r) * out_stride;
#pragma unroll
    for (int w = 0; w < WORDS; ++w) o[w] = mine[w];
  }
}

// ------------------------------------------------------------------------------------------------ decode step

struct DecodeArgs {
  he_config cfg;
  he_cache ca;
  const void* q;
  const void* k;
  const void* v;
  int32_t* victim_out;
  int32_t* evicted_pos_out;
  uint32_t* qcodes_out;
};

constexpr int kRowBatch = 5;    // rows hashed per pass in the decode kernel (G = 4 queries + the key)
constexpr int kDecodeVecs = 8;  // 16-byte code vectors held in registers per thread

template <int WORDS, int GT>
__device__ __forceinline__ int group_distance(uint32_t c0, uint32_t c1, const uint32_t (&qreg)[GT > 0 ? GT : 1][WORDS],
                                              const uint32_t* qsm, int G) {
  int D = 0;
  if (GT > 0) {
#pragma unroll
    for (int g = 0; g < GT; ++g) {
      D += __popc(c0 ^ qreg[g][0]);
      if (WORDS == 2) D += __popc(c1 ^ qreg[g][WORDS - 1]);
    }
  } else {
    for (int g = 0; g < G; ++g) {
      D += __popc(c0 ^ qsm[g * WORDS]);
      if (WORDS == 2) D += __popc(c1 ^ qsm[g * WORDS + WORDS - 1]);
    }
  }
  return D;
}

template <int WORDS, int GT, int NT>
__global__ void __launch_bounds__(NT) decode_step_kernel(const DecodeArgs a) {
  constexpr int SPV = 4 / WORDS;  // slots per 16-byte vector
  constexpr int BP = 32 * WORDS;
  __shared__ __align__(16) float xs[kRowBatch][kMaxDim];
  __shared__ float part[kMaxDim / kChunk][kRowBatch][BP];
  __shared__ uint32_t codes_s[(kMaxGroup + 1) * WORDS];  // rows 0..G-1: query codes, row G: key code
  __shared__ uint32_t wbest[2][32];

  const he_config& cfg = a.cfg;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long unit = blockIdx.x;
  const int s = (int)(unit / cfg.n_kv_heads);
  const int d = cfg.head_dim, b = cfg.hash_bits, G = cfg.group_size, es = esize_of(cfg.dtype);
  const long long Cmax = cfg.max_budget;
  const int C = a.ca.budget[s];
  const int fill = a.ca.fill[unit];
  const int t = a.ca.next_pos[unit];
  const bool evict = fill >= C;

  // (1) pull this unit's code words into registers; they are in flight while the new rows are hashed
  uint4 cv[kDecodeVecs];
  const uint4* cvec = reinterpret_cast<const uint4*>(a.ca.codes + unit * Cmax * WORDS);
  const int nvec = evict ? (C * WORDS + 3) / 4 : 0;
#pragma unroll
  for (int i = 0; i < kDecodeVecs; ++i) {
    const int vi = i * NT + tid;
    cv[i] = vi < nvec ? __ldg(cvec + vi) : make_uint4(0u, 0u, 0u, 0u);
  }
  // the new K and V rows, 16 bytes per thread, kept until the victim is known
  const int cpr = d * es / 16;
  uint4 rowreg = make_uint4(0u, 0u, 0u, 0u);
  if (tid < 2 * cpr) {
    const char* src = static_cast<const char*>(tid < cpr ? a.k : a.v) + unit * d * es;
    rowreg = __ldg(reinterpret_cast<const uint4*>(src) + (tid % cpr));
  }

  // (2) hash the G query rows and the key row (Eq. 2)
  const int R = G + 1;
  const int nch = (d + kChunk - 1) / kChunk;
  for (int r0 = 0; r0 < R; r0 += kRowBatch) {
    for (int idx = tid; idx < kRowBatch * cpr; idx += NT) {
      const int r = idx / cpr, ch = idx % cpr, row = r0 + r;
      if (row < R) {
        const char* src = row < G ? static_cast<const char*>(a.q) + (unit * G + row) * d * es
                                  : static_cast<const char*>(a.k) + unit * d * es;
        stage_chunk(xs[r], src, ch, cfg.dtype);
      } else {
        for (int i = 0; i < 16 / es; ++i) xs[r][ch * (16 / es) + i] = 0.f;
      }
    }
    __syncthreads();
    for (int item = tid; item < nch * BP; item += NT) {
      const int qd = item / BP, i = item % BP;
      float acc[kRowBatch];
#pragma unroll
      for (int r = 0; r < kRowBatch; ++r) acc[r] = 0.f;
      const int c0 = qd * kChunk;
      const int cend = (d - c0) < kChunk ? (d - c0) : kChunk;
      if (i < b) {
#pragma unroll 8
        for (int cc = 0; cc < cend; ++cc) {
          const float wv = __ldg(a.ca.W + (long long)(c0 + cc) * b + i);
#pragma unroll
          for (int r = 0; r < kRowBatch; ++r) acc[r] = fmaf(xs[r][c0 + cc], wv, acc[r]);
        }
      }
#pragma unroll
      for (int r = 0; r < kRowBatch; ++r) part[qd][r][i] = acc[r];
    }
    __syncthreads();
    for (int task = warp; task < kRowBatch * WORDS; task += NT / 32) {
      const int r = task / WORDS, w = task % WORDS;
      float tot = 0.f;
      for (int qd = 0; qd < nch; ++qd) tot += part[qd][r][w * 32 + lane];
      const uint32_t word = __ballot_sync(0xFFFFFFFFu, tot >= 0.f) & word_mask(b, w);
      if (lane == 0 && r0 + r < R) codes_s[(r0 + r) * WORDS + w] = word;
    }
    __syncthreads();
  }
  if (a.qcodes_out != nullptr && tid < G * WORDS) a.qcodes_out[unit * G * WORDS + tid] = codes_s[tid];

  // (3) Eq. 5 / Eq. 6: Hamming distance of every slot to the query codes, arg-max with lowest-index ties
  int slot = fill;
  if (evict) {
    uint32_t qreg[GT > 0 ? GT : 1][WORDS];
    if (GT > 0) {
#pragma unroll
      for (int g = 0; g < GT; ++g)
#pragma unroll
        for (int w = 0; w < WORDS; ++w) qreg[g][w] = codes_s[g * WORDS + w];
    }
    const bool prot = cfg.n_sink > 0 || cfg.n_recent > 0;
    const bool write_scores = (cfg.flags & HE_FLAG_WRITE_SCORES) != 0;
    float* sc = a.ca.scores + unit * Cmax;
    const int32_t* pp = a.ca.pos + unit * Cmax;
    uint32_t best_all = 0u, best_el = 0u;
#pragma unroll
    for (int i = 0; i < kDecodeVecs; ++i) {
      const int vi = i * NT + tid;
      if (vi < nvec) {
        const int j0 = vi * SPV;
        const uint32_t wds[4] = {cv[i].x, cv[i].y, cv[i].z, cv[i].w};
        float sv[SPV];
#pragma unroll
        for (int e = 0; e < SPV; ++e) {
          const int j = j0 + e;
          const int D = group_distance<WORDS, GT>(wds[e * WORDS], wds[e * WORDS + WORDS - 1], qreg, codes_s, G);
          sv[e] = -(float)D;
          if (j < C) {
            const uint32_t key = ((uint32_t)(D + 1) << kKeyIdxBits) | (kKeyIdxMask - (uint32_t)j);
            best_all = max(best_all, key);
            if (prot) {
              const int p = __ldg(pp + j);
              if (p >= cfg.n_sink && p < t - cfg.n_recent) best_el = max(best_el, key);
            }
          }
        }
        if (write_scores) {
          if (j0 + SPV <= C) {
            if (SPV == 4) *reinterpret_cast<float4*>(sc + j0) = make_float4(sv[0], sv[1], sv[SPV > 2 ? 2 : 0], sv[SPV > 3 ? 3 : 0]);
            else *reinterpret_cast<float2*>(sc + j0) = make_float2(sv[0], sv[1]);
          } else {
#pragma unroll
            for (int e = 0; e < SPV; ++e)
              if (j0 + e < C) sc[j0 + e] = sv[e];
          }
        }
      }
    }
    best_all = __reduce_max_sync(0xFFFFFFFFu, best_all);
    if (prot) best_el = __reduce_max_sync(0xFFFFFFFFu, best_el);
    if (lane == 0) {
      wbest[0][warp] = best_all;
      wbest[1][warp] = best_el;
    }
    __syncthreads();
    uint32_t fin = __reduce_max_sync(0xFFFFFFFFu, lane < NT / 32 ? wbest[0][lane] : 0u);
    if (prot) {
      const uint32_t fin_el = __reduce_max_sync(0xFFFFFFFFu, lane < NT / 32 ? wbest[1][lane] : 0u);
      if (fin_el != 0u) fin = fin_el;
    }
    slot = (int)(kKeyIdxMask - (fin & kKeyIdxMask));
  }

  // (4) Algorithm 1 lines 2-5: the slot takes the new token's K, V, code and position
  if (tid < 2 * cpr) {
    char* dst = static_cast<char*>(tid < cpr ? a.ca.k_cache : a.ca.v_cache) + (unit * Cmax + slot) * d * es;
    reinterpret_cast<uint4*>(dst)[tid % cpr] = rowreg;
  }
  if (tid == NT - 1) {
    int ev = -1;
    if (evict && a.evicted_pos_out != nullptr) ev = a.ca.pos[unit * Cmax + slot];
    a.ca.pos[unit * Cmax + slot] = t;
#pragma unroll
    for (int w = 0; w < WORDS; ++w) a.ca.codes[(unit * Cmax + slot) * WORDS + w] = codes_s[G * WORDS + w];
    if (!evict) {
      a.ca.scores[unit * Cmax + slot] = 0.f;
      a.ca.fill[unit] = fill + 1;
    }
    a.ca.next_pos[unit] = t + 1;
    a.victim_out[unit] = slot;
    if (a.evicted_pos_out != nullptr) a.evicted_pos_out[unit] = ev;
  }
}

// ------------------------------------------------------------------------------------------------ prefill replay

struct ReplayArgs {
  he_config cfg;
  he_cache ca;
  const uint32_t* kcodes;  // [units, Nmax, Wd]
  const uint32_t* qcodes;  // [units, Nmax, G, Wd]
  const int32_t* prompt_len;
  long long Nmax;
  int smem_slots;  // slots the shared-memory tables were sized for
};

constexpr int kStepBlock = 32;  // prompt tokens whose codes are staged in shared memory at a time
constexpr int kPrefMax = 5;     // staged words per thread, enough for 32 * 9 * 2 words on 128 threads

template <int WORDS, int GT>
__global__ void prefill_replay_kernel(const ReplayArgs a) {
  extern __shared__ __align__(16) uint32_t rsm[];
  __shared__ uint32_t wbest[2][2][32];
  __shared__ uint32_t stage[2][kStepBlock * (kMaxGroup + 1) * WORDS];

  const he_config& cfg = a.cfg;
  const int NT = blockDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = NT >> 5;
  const long long unit = blockIdx.x;
  const int s = (int)(unit / cfg.n_kv_heads);
  const int G = cfg.group_size;
  const long long Cmax = cfg.max_budget;
  const int C = a.ca.budget[s];
  const int N = a.prompt_len[s];
  const int fill0 = N < C ? N : C;
  uint32_t* codes_s = rsm;                                      // [smem_slots][WORDS]
  int32_t* pos_s = reinterpret_cast<int32_t*>(rsm + (size_t)a.smem_slots * WORDS);  // [smem_slots]
  const uint32_t* kc_u = a.kcodes + unit * a.Nmax * WORDS;
  const uint32_t* qc_u = a.qcodes + unit * a.Nmax * G * WORDS;
  const bool prot = cfg.n_sink > 0 || cfg.n_recent > 0;
  const bool write_scores = (cfg.flags & HE_FLAG_WRITE_SCORES) != 0;
  float* sc = a.ca.scores + unit * Cmax;

  // first C tokens fill the cache in order (Section 3, "Prompt Encoding Stage")
  for (int j = tid; j < fill0; j += NT) {
#pragma unroll
    for (int w = 0; w < WORDS; ++w) codes_s[j * WORDS + w] = kc_u[(long long)j * WORDS + w];
    pos_s[j] = j;
  }

  // codes of the next kStepBlock tokens: query part then key part
  const int qwords = G * WORDS;
  const int stage_words = kStepBlock * (qwords + WORDS);
  uint32_t pref[kPrefMax];
  auto prefetch = [&](int t0) {
#pragma unroll
    for (int i = 0; i < kPrefMax; ++i) {
      const int e = i * NT + tid;
      uint32_t val = 0u;
      if (e < stage_words) {
        if (e < kStepBlock * qwords) {
          const long long tt = t0 + e / qwords;
          if (tt < N) val = __ldg(qc_u + (long long)t0 * qwords + e);
        } else {
          const int e2 = e - kStepBlock * qwords;
          const long long tt = t0 + e2 / WORDS;
          if (tt < N) val = __ldg(kc_u + (long long)t0 * WORDS + e2);
        }
      }
      pref[i] = val;
    }
  };
  auto commit = [&](int buf) {
#pragma unroll
    for (int i = 0; i < kPrefMax; ++i) {
      const int e = i * NT + tid;
      if (e < stage_words) stage[buf][e] = pref[i];
    }
  };

  int buf = 0;
  if (C < N) {
    prefetch(C);
    commit(0);
  }
  __syncthreads();

  int par = 0;
  for (int t0 = C; t0 < N; t0 += kStepBlock) {
    const bool more = t0 + kStepBlock < N;
    if (more) prefetch(t0 + kStepBlock);
    const int tend = (N - t0) < kStepBlock ? (N - t0) : kStepBlock;
    for (int ts = 0; ts < tend; ++ts) {
      const int t = t0 + ts;
      const uint32_t* qsm = &stage[buf][ts * qwords];
      uint32_t qreg[GT > 0 ? GT : 1][WORDS];
      if (GT > 0) {
#pragma unroll
        for (int g = 0; g < GT; ++g)
#pragma unroll
          for (int w = 0; w < WORDS; ++w) qreg[g][w] = qsm[g * WORDS + w];
      }
      const bool last = write_scores && (t == N - 1);
      uint32_t best_all = 0u, best_el = 0u;
      for (int j = tid; j < C; j += NT) {
        uint32_t c0, c1 = 0u;
        if (WORDS == 2) {
          const uint2 cc = *reinterpret_cast<const uint2*>(codes_s + j * 2);
          c0 = cc.x;
          c1 = cc.y;
        } else {
          c0 = codes_s[j];
        }
        const int D = group_distance<WORDS, GT>(c0, c1, qreg, qsm, G);
        const uint32_t key = ((uint32_t)(D + 1) << kKeyIdxBits) | (kKeyIdxMask - (uint32_t)j);
        best_all = max(best_all, key);
        if (prot) {
          const int p = pos_s[j];
          if (p >= cfg.n_sink && p < t - cfg.n_recent) best_el = max(best_el, key);
        }
        if (last) sc[j] = -(float)D;
      }
      best_all = __reduce_max_sync(0xFFFFFFFFu, best_all);
      if (prot) best_el = __reduce_max_sync(0xFFFFFFFFu, best_el);
      if (lane == 0) {
        wbest[par][0][warp] = best_all;
        wbest[par][1][warp] = best_el;
      }
      __syncthreads();
      uint32_t fin = __reduce_max_sync(0xFFFFFFFFu, lane < nwarps ? wbest[par][0][lane] : 0u);
      if (prot) {
        const uint32_t fin_el = __reduce_max_sync(0xFFFFFFFFu, lane < nwarps ? wbest[par][1][lane] : 0u);
        if (fin_el != 0u) fin = fin_el;
      }
      const int slot = (int)(kKeyIdxMask - (fin & kKeyIdxMask));
      if (slot % NT == tid) {  // the slot's own scanning thread rewrites it, so no extra barrier is needed
#pragma unroll
        for (int w = 0; w < WORDS; ++w) codes_s[slot * WORDS + w] = stage[buf][kStepBlock * qwords + ts * WORDS + w];
        pos_s[slot] = t;
      }
      par ^= 1;
    }
    if (more) {
      commit(buf ^ 1);
      __syncthreads();
      buf ^= 1;
    }
  }
  __syncthreads();

  // final state of the unit; everything beyond `fill` is reset
  const bool scored = write_scores && N > C;
  for (int j = tid; j < Cmax; j += NT) {
    const bool valid = j < fill0;
#pragma unroll
    for (int w = 0; w < WORDS; ++w) a.ca.codes[(unit * Cmax + j) * WORDS + w] = valid ? codes_s[j * WORDS + w] : 0u;
    a.ca.pos[unit * Cmax + j] = valid ? pos_s[j] : -1;
    if (!(valid && scored)) sc[j] = 0.f;
  }
  if (tid == 0) {
    a.ca.fill[unit] = fill0;
    a.ca.next_pos[unit] = N;
  }
}

// ------------------------------------------------------------------------------------------------ prefill gather

struct GatherArgs {
  he_config cfg;
  he_cache ca;
  const void* k;
  const void* v;
  long long s0, s1, s2;
};

constexpr int kGatherThreads = 256;
constexpr int kGatherUnroll = 4;

__global__ void __launch_bounds__(kGatherThreads) prefill_gather_kernel(const GatherArgs a) {
  const he_config& cfg = a.cfg;
  const long long unit = blockIdx.y;
  const int s = (int)(unit / cfg.n_kv_heads), h = (int)(unit % cfg.n_kv_heads);
  const int d = cfg.head_dim, es = esize_of(cfg.dtype);
  const long long Cmax = cfg.max_budget;
  const int fill = a.ca.fill[unit];
  const int cpr = d * es / 16;
  const long long ntask = 2LL * fill * cpr;
  const long long base = (long long)blockIdx.x * kGatherThreads * kGatherUnroll;
  if (base >= ntask) return;
  const int32_t* pp = a.ca.pos + unit * Cmax;
  uint4 val[kGatherUnroll];
  long long dst_off[kGatherUnroll];
#pragma unroll
  for (int i = 0; i < kGatherUnroll; ++i) {
    const long long task = base + (long long)i * kGatherThreads + threadIdx.x;
    dst_off[i] = -1;
    if (task < ntask) {
      const int which = (int)(task / ((long long)fill * cpr));
      const long long rem = task % ((long long)fill * cpr);
      const int j = (int)(rem / cpr), ch = (int)(rem % cpr);
      const long long tok = pp[j];
      const char* src = static_cast<const char*>(which ? a.v : a.k) + (s * a.s0 + h * a.s1 + tok * a.s2) * es;
      val[i] = __ldg(reinterpret_cast<const uint4*>(src) + ch);
      dst_off[i] = (((unit * Cmax + j) * d * es) / 16 + ch) * 2 + which;
    }
  }
#pragma unroll
  for (int i = 0; i < kGatherUnroll; ++i)
    if (dst_off[i] >= 0) {
      uint4* dst = reinterpret_cast<uint4*>((dst_off[i] & 1) ? a.ca.v_cache : a.ca.k_cache);
      dst[dst_off[i] >> 1] = val[i];
    }
}

// ------------------------------------------------------------------------------------------------ reset

__global__ void reset_kernel(const he_config cfg, const he_cache ca) {
  const long long units = (long long)cfg.batch * cfg.n_kv_heads;
  const long long slots = units * cfg.max_budget;
  const int Wd = words_of(cfg.hash_bits);
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < slots; i += stride) {
    ca.pos[i] = -1;
    ca.scores[i] = 0.f;
    for (int w = 0; w < Wd; ++w) ca.codes[i * Wd + w] = 0u;
    if (i < units) {
      ca.fill[i] = 0;
      ca.next_pos[i] = 0;
    }
  }
}

// ------------------------------------------------------------------------------------------------ host side

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_config(const he_config* cfg, bool need_cache_dims) {
  if (cfg == nullptr) return fail(HE_ERR_INVALID_ARG, "cfg is null");
  if (cfg->dtype != HE_DTYPE_F32 && cfg->dtype != HE_DTYPE_BF16) return fail(HE_ERR_INVALID_ARG, "dtype %d is not HE_DTYPE_F32/BF16", cfg->dtype);
  if (cfg->hash_bits < 1 || cfg->hash_bits > 64) return fail(HE_ERR_INVALID_ARG, "hash_bits %d outside [1, 64]", cfg->hash_bits);
  if (cfg->head_dim < 8 || cfg->head_dim % 8 != 0) return fail(HE_ERR_INVALID_ARG, "head_dim %d is not a positive multiple of 8", cfg->head_dim);
  if (cfg->head_dim > kMaxDim) return fail(HE_ERR_UNSUPPORTED, "head_dim %d > %d", cfg->head_dim, kMaxDim);
  if (!need_cache_dims) return HE_OK;
  if (cfg->batch < 1 || cfg->n_kv_heads < 1) return fail(HE_ERR_INVALID_ARG, "batch %d / n_kv_heads %d must be >= 1", cfg->batch, cfg->n_kv_heads);
  if (cfg->group_size < 1) return fail(HE_ERR_INVALID_ARG, "group_size %d must be >= 1", cfg->group_size);
  if (cfg->group_size > kMaxGroup) return fail(HE_ERR_UNSUPPORTED, "group_size %d > %d", cfg->group_size, kMaxGroup);
  if (cfg->max_budget < 4 || cfg->max_budget % 4 != 0) return fail(HE_ERR_INVALID_ARG, "max_budget %d is not a positive multiple of 4", cfg->max_budget);
  if (cfg->max_budget > (1 << kKeyIdxBits)) return fail(HE_ERR_UNSUPPORTED, "max_budget %d > 2^20", cfg->max_budget);
  if (cfg->n_sink < 0 || cfg->n_recent < 0) return fail(HE_ERR_INVALID_ARG, "n_sink / n_recent must be >= 0");
  return HE_OK;
}

int check_cache(const he_cache* ca) {
  if (ca == nullptr) return fail(HE_ERR_INVALID_ARG, "cache is null");
  if (!ca->k_cache || !ca->v_cache || !ca->codes || !ca->scores || !ca->pos || !ca->budget || !ca->fill || !ca->next_pos || !ca->W)
    return fail(HE_ERR_INVALID_ARG, "cache has a null pointer");
  if (!aligned16(ca->k_cache) || !aligned16(ca->v_cache) || !aligned16(ca->codes) || !aligned16(ca->scores) || !aligned16(ca->pos))
    return fail(HE_ERR_INVALID_ARG, "cache arrays must be 16-byte aligned");
  return HE_OK;
}

template <typename K>
int set_smem(K kernel, size_t bytes) {
  if (bytes > 48 * 1024) HE_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
  return HE_OK;
}

int launch_hash(const HashJob& job, long long max_rows_per_segment, int segments, cudaStream_t stream) {
  if (max_rows_per_segment <= 0 || segments <= 0) return HE_OK;
  const int Wd = words_of(job.b);
  const size_t smem = ((size_t)job.d * 32 * Wd + (size_t)kHashRows * job.d) * sizeof(float);
  const long long tiles = (max_rows_per_segment + kHashRows - 1) / kHashRows;
  if (tiles > 0x7FFFFFFFLL || segments > 65535) return fail(HE_ERR_UNSUPPORTED, "hash grid too large (%lld x %d)", tiles, segments);
  dim3 grid((unsigned)tiles, (unsigned)segments);
  if (Wd == 1) {
    if (int rc = set_smem(hash_rows_kernel<1>, smem)) return rc;
    hash_rows_kernel<1><<<grid, kHashThreads, smem, stream>>>(job);
  } else {
    if (int rc = set_smem(hash_rows_kernel<2>, smem)) return rc;
    hash_rows_kernel<2><<<grid, kHashThreads, smem, stream>>>(job);
  }
  HE_CUDA_CHECK(cudaGetLastError());
  return HE_OK;
}

template <int WORDS, int GT>
int launch_decode_nt(const DecodeArgs& a, int nt, long long units, cudaStream_t stream) {
  if (nt == 256) decode_step_kernel<WORDS, GT, 256><<<(unsigned)units, 256, 0, stream>>>(a);
  else if (nt == 512) decode_step_kernel<WORDS, GT, 512><<<(unsigned)units, 512, 0, stream>>>(a);
  else decode_step_kernel<WORDS, GT, 1024><<<(unsigned)units, 1024, 0, stream>>>(a);
  HE_CUDA_CHECK(cudaGetLastError());
  return HE_OK;
}

template <int WORDS>
int launch_decode_g(const DecodeArgs& a, int nt, long long units, cudaStream_t stream) {
  switch (a.cfg.group_size) {
    case 1: return launch_decode_nt<WORDS, 1>(a, nt, units, stream);
    case 4: return launch_decode_nt<WORDS, 4>(a, nt, units, stream);
    default: return launch_decode_nt<WORDS, 0>(a, nt, units, stream);
  }
}

template <int WORDS, int GT>
int launch_replay_one(const ReplayArgs& a, int nt, size_t smem, long long units, cudaStream_t stream) {
  if (int rc = set_smem(prefill_replay_kernel<WORDS, GT>, smem)) return rc;
  prefill_replay_kernel<WORDS, GT><<<(unsigned)units, nt, smem, stream>>>(a);
  HE_CUDA_CHECK(cudaGetLastError());
  return HE_OK;
}

template <int WORDS>
int launch_replay_g(const ReplayArgs& a, int nt, size_t smem, long long units, cudaStream_t stream) {
  switch (a.cfg.group_size) {
    case 1: return launch_replay_one<WORDS, 1>(a, nt, smem, units, stream);
    case 4: return launch_replay_one<WORDS, 4>(a, nt, smem, units, stream);
    default: return launch_replay_one<WORDS, 0>(a, nt, smem, units, stream);
  }
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace

extern "C" {

const char* he_last_error(void) { return g_err; }

int he_hash_keys(const he_config* cfg, const void* x, int64_t rows, int64_t row_stride_elems, const float* W,
                 uint32_t* codes_out, void* stream) {
  if (int rc = check_config(cfg, false)) return rc;
  if (rows < 0) return fail(HE_ERR_INVALID_ARG, "rows %lld < 0", (long long)rows);
  if (rows == 0) return HE_OK;
  if (!x || !W || !codes_out) return fail(HE_ERR_INVALID_ARG, "x, W or codes_out is null");
  const int es = esize_of(cfg->dtype);
  if (row_stride_elems < cfg->head_dim || (row_stride_elems * es) % 16 != 0 || !aligned16(x))
    return fail(HE_ERR_INVALID_ARG, "rows of x must be 16-byte aligned with a stride >= head_dim");
  HashJob job{};
  job.x = x;
  job.W = W;
  job.out = codes_out;
  job.mode = 0;
  job.dtype = cfg->dtype;
  job.d = cfg->head_dim;
  job.b = cfg->hash_bits;
  job.rows = rows;
  job.row_stride = row_stride_elems;
  return launch_hash(job, rows, 1, static_cast<cudaStream_t>(stream));
}

int he_decode_step(const he_config* cfg, const he_cache* cache, const void* q, const void* k, const void* v,
                   int32_t* victim_out, int32_t* evicted_pos_out, uint32_t* qcodes_out, void* stream) {
  if (int rc = check_config(cfg, true)) return rc;
  if (int rc = check_cache(cache)) return rc;
  if (!q || !k || !v || !victim_out) return fail(HE_ERR_INVALID_ARG, "q, k, v or victim_out is null");
  if (!aligned16(q) || !aligned16(k) || !aligned16(v)) return fail(HE_ERR_INVALID_ARG, "q, k, v must be 16-byte aligned");
  const int Wd = words_of(cfg->hash_bits);
  const long long nvec = ((long long)cfg->max_budget * Wd + 3) / 4;
  int nt = 256;
  if (nvec > 256LL * kDecodeVecs) nt = 512;
  if (nvec > 512LL * kDecodeVecs) nt = 1024;
  if (nvec > 1024LL * kDecodeVecs)
    return fail(HE_ERR_UNSUPPORTED, "max_budget %d with %d code words exceeds the decode kernel's %d slots", cfg->max_budget, Wd,
                1024 * kDecodeVecs * 4 / Wd);
  const long long units = (long long)cfg->batch * cfg->n_kv_heads;
  if (units > 0x7FFFFFFFLL) return fail(HE_ERR_UNSUPPORTED, "too many units");
  DecodeArgs a{*cfg, *cache, q, k, v, victim_out, evicted_pos_out, qcodes_out};
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return Wd == 1 ? launch_decode_g<1>(a, nt, units, st) : launch_decode_g<2>(a, nt, units, st);
}

size_t he_workspace_bytes(const he_config* cfg, int32_t max_prompt_len) {
  if (check_config(cfg, true) != HE_OK || max_prompt_len < 0) return 0;
  const size_t units = (size_t)cfg->batch * cfg->n_kv_heads;
  const size_t Wd = words_of(cfg->hash_bits);
  const size_t kbytes = align_up(units * (size_t)max_prompt_len * Wd * 4, 256);
  const size_t qbytes = align_up(units * (size_t)max_prompt_len * cfg->group_size * Wd * 4, 256);
  return kbytes + qbytes + 256;
}

int he_prefill_compress(const he_config* cfg, const he_cache* cache, const void* q, const void* k, const void* v,
                        const int64_t q_strides[3], const int64_t kv_strides[3], const int32_t* prompt_len,
                        int32_t max_prompt_len, void* workspace, size_t workspace_bytes, void* stream) {
  if (int rc = check_config(cfg, true)) return rc;
  if (int rc = check_cache(cache)) return rc;
  if (!q || !k || !v || !q_strides || !kv_strides || !prompt_len || !workspace)
    return fail(HE_ERR_INVALID_ARG, "q, k, v, strides, prompt_len or workspace is null");
  if (max_prompt_len < 0) return fail(HE_ERR_INVALID_ARG, "max_prompt_len %d < 0", max_prompt_len);
  const int es = esize_of(cfg->dtype);
  for (int i = 0; i < 3; ++i)
    if ((q_strides[i] * es) % 16 != 0 || (kv_strides[i] * es) % 16 != 0)
      return fail(HE_ERR_INVALID_ARG, "strides must keep every row 16-byte aligned");
  if (!aligned16(q) || !aligned16(k) || !aligned16(v)) return fail(HE_ERR_INVALID_ARG, "q, k, v must be 16-byte aligned");
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return fail(HE_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
  const size_t need = he_workspace_bytes(cfg, max_prompt_len);
  if (workspace_bytes < need) return fail(HE_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, need);

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const long long units = (long long)cfg->batch * cfg->n_kv_heads;
  const int Wd = words_of(cfg->hash_bits), G = cfg->group_size;
  uint32_t* kcodes = static_cast<uint32_t*>(workspace);
  uint32_t* qcodes = reinterpret_cast<uint32_t*>(static_cast<char*>(workspace) +
                                                 align_up((size_t)units * max_prompt_len * Wd * 4, 256));

  // phase 1: Eq. 2 on every prompt key and on the queries of the tokens that will evict
  HashJob job{};
  job.W = cache->W;
  job.dtype = cfg->dtype;
  job.d = cfg->head_dim;
  job.b = cfg->hash_bits;
  job.Hkv = cfg->n_kv_heads;
  job.G = G;
  job.Nmax = max_prompt_len;
  job.prompt_len = prompt_len;
  job.budget = cache->budget;
  job.x = k;
  job.out = kcodes;
  job.mode = 1;
  job.heads = cfg->n_kv_heads;
  job.s0 = kv_strides[0];
  job.s1 = kv_strides[1];
  job.s2 = kv_strides[2];
  if (int rc = launch_hash(job, max_prompt_len, (int)units, st)) return rc;
  job.x = q;
  job.out = qcodes;
  job.mode = 2;
  job.heads = cfg->n_kv_heads * G;
  job.s0 = q_strides[0];
  job.s1 = q_strides[1];
  job.s2 = q_strides[2];
  if (int rc = launch_hash(job, max_prompt_len, (int)units * G, st)) return rc;

  // phase 2: the sequential replay of Algorithm 1 over the prompt, one CTA per unit
  ReplayArgs ra{*cfg, *cache, kcodes, qcodes, prompt_len, max_prompt_len, cfg->max_budget};
  const size_t smem = (size_t)cfg->max_budget * (Wd + 1) * 4;
  if (smem > 200 * 1024) return fail(HE_ERR_UNSUPPORTED, "max_budget %d does not fit the replay kernel's shared memory", cfg->max_budget);
  int nt = 256;
  if (cfg->max_budget > 4096) nt = 512;
  if (cfg->max_budget > 16384) nt = 1024;
  if (int rc = (Wd == 1 ? launch_replay_g<1>(ra, nt, smem, units, st) : launch_replay_g<2>(ra, nt, smem, units, st))) return rc;

  // phase 3: surviving K / V rows into their slots
  GatherArgs ga{*cfg, *cache, k, v, kv_strides[0], kv_strides[1], kv_strides[2]};
  const long long per_unit = 2LL * cfg->max_budget * (cfg->head_dim * es / 16);
  const long long gx = (per_unit + kGatherThreads * kGatherUnroll - 1) / (kGatherThreads * kGatherUnroll);
  if (units > 65535) return fail(HE_ERR_UNSUPPORTED, "more than 65535 units in one prefill call");
  prefill_gather_kernel<<<dim3((unsigned)gx, (unsigned)units), kGatherThreads, 0, st>>>(ga);
  HE_CUDA_CHECK(cudaGetLastError());
  return HE_OK;
}

int he_reset(const he_config* cfg, const he_cache* cache, void* stream) {
  if (int rc = check_config(cfg, true)) return rc;
  if (int rc = check_cache(cache)) return rc;
  const long long slots = (long long)cfg->batch * cfg->n_kv_heads * cfg->max_budget;
  const int blocks = (int)((slots + 255) / 256 < 148 * 8 ? (slots + 255) / 256 : 148 * 8);
  reset_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(*cfg, *cache);
  HE_CUDA_CHECK(cudaGetLastError());
  return HE_OK;
}

size_t he_decode_staging_bytes(const he_config* cfg) {
  if (check_config(cfg, true) != HE_OK) return 0;
  const size_t units = (size_t)cfg->batch * cfg->n_kv_heads;
  const size_t row = (size_t)cfg->head_dim * esize_of(cfg->dtype);
  return align_up(units * cfg->group_size * row, 256) + 2 * align_up(units * row, 256) + align_up(units * 4, 256);
}

int he_decode_step_host(const he_config* cfg, const he_cache* cache, const void* q_host, const void* k_host,
                        const void* v_host, int32_t* victim_host, void* staging, size_t staging_bytes, void* stream) {
  if (int rc = check_config(cfg, true)) return rc;
  if (!q_host || !k_host || !v_host || !victim_host || !staging) return fail(HE_ERR_INVALID_ARG, "a host pointer or staging is null");
  if ((reinterpret_cast<uintptr_t>(staging) & 255u) != 0) return fail(HE_ERR_INVALID_ARG, "staging must be 256-byte aligned");
  const size_t need = he_decode_staging_bytes(cfg);
  if (staging_bytes < need) return fail(HE_ERR_WORKSPACE, "staging has %zu bytes, %zu needed", staging_bytes, need);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t units = (size_t)cfg->batch * cfg->n_kv_heads;
  const size_t row = (size_t)cfg->head_dim * esize_of(cfg->dtype);
  char* p = static_cast<char*>(staging);
  void* dq = p;
  p += align_up(units * cfg->group_size * row, 256);
  void* dk = p;
  p += align_up(units * row, 256);
  void* dv = p;
  p += align_up(units * row, 256);
  int32_t* dvictim = reinterpret_cast<int32_t*>(p);
  HE_CUDA_CHECK(cudaMemcpyAsync(dq, q_host, units * cfg->group_size * row, cudaMemcpyHostToDevice, st));
  HE_CUDA_CHECK(cudaMemcpyAsync(dk, k_host, units * row, cudaMemcpyHostToDevice, st));
  HE_CUDA_CHECK(cudaMemcpyAsync(dv, v_host, units * row, cudaMemcpyHostToDevice, st));
  if (int rc = he_decode_step(cfg, cache, dq, dk, dv, dvictim, nullptr, nullptr, stream)) return rc;
  HE_CUDA_CHECK(cudaMemcpyAsync(victim_host, dvictim, units * 4, cudaMemcpyDeviceToHost, st));
  HE_CUDA_CHECK(cudaStreamSynchronize(st));
  return HE_OK;
}

size_t he_prefill_staging_bytes(const he_config* cfg, int32_t max_prompt_len) {
  const size_t ws = he_workspace_bytes(cfg, max_prompt_len);
  if (ws == 0) return 0;
  const size_t units = (size_t)cfg->batch * cfg->n_kv_heads;
  const size_t rows = units * (size_t)max_prompt_len * cfg->head_dim * esize_of(cfg->dtype);
  return align_up(ws, 256) + align_up(rows * cfg->group_size, 256) + 2 * align_up(rows, 256) + align_up((size_t)cfg->batch * 4, 256);
}

int he_prefill_compress_host(const he_config* cfg, const he_cache* cache, const void* q_host, const void* k_host,
                             const void* v_host, const int32_t* prompt_len_host, int32_t max_prompt_len,
                             int32_t* fill_host, void* staging, size_t staging_bytes, void* stream) {
  if (int rc = check_config(cfg, true)) return rc;
  if (int rc = check_cache(cache)) return rc;
  if (!q_host || !k_host || !v_host || !prompt_len_host || !fill_host || !staging) return fail(HE_ERR_INVALID_ARG, "a host pointer or staging is null");
  if ((reinterpret_cast<uintptr_t>(staging) & 255u) != 0) return fail(HE_ERR_INVALID_ARG, "staging must be 256-byte aligned");
  if (max_prompt_len < 0) return fail(HE_ERR_INVALID_ARG, "max_prompt_len %d < 0", max_prompt_len);
  const size_t need = he_prefill_staging_bytes(cfg, max_prompt_len);
  if (staging_bytes < need) return fail(HE_ERR_WORKSPACE, "staging has %zu bytes, %zu needed", staging_bytes, need);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t units = (size_t)cfg->batch * cfg->n_kv_heads;
  const size_t rows = units * (size_t)max_prompt_len * cfg->head_dim * esize_of(cfg->dtype);
  const size_t ws = he_workspace_bytes(cfg, max_prompt_len);
  char* p = static_cast<char*>(staging);
  void* dws = p;
  p += align_up(ws, 256);
  void* dq = p;
  p += align_up(rows * cfg->group_size, 256);
  void* dk = p;
  p += align_up(rows, 256);
  void* dv = p;
  p += align_up(rows, 256);
  int32_t* dlen = reinterpret_cast<int32_t*>(p);
  HE_CUDA_CHECK(cudaMemcpyAsync(dq, q_host, rows * cfg->group_size, cudaMemcpyHostToDevice, st));
  HE_CUDA_CHECK(cudaMemcpyAsync(dk, k_host, rows, cudaMemcpyHostToDevice, st));
  HE_CUDA_CHECK(cudaMemcpyAsync(dv, v_host, rows, cudaMemcpyHostToDevice, st));
  HE_CUDA_CHECK(cudaMemcpyAsync(dlen, prompt_len_host, (size_t)cfg->batch * 4, cudaMemcpyHostToDevice, st));
  const int64_t N = max_prompt_len, d = cfg->head_dim;
  const int64_t qs[3] = {(int64_t)cfg->n_kv_heads * cfg->group_size * N * d, N * d, d};
  const int64_t ks[3] = {(int64_t)cfg->n_kv_heads * N * d, N * d, d};
  if (int rc = he_prefill_compress(cfg, cache, dq, dk, dv, qs, ks, dlen, max_prompt_len, dws, ws, stream)) return rc;
  HE_CUDA_CHECK(cudaMemcpyAsync(fill_host, cache->fill, units * 4, cudaMemcpyDeviceToHost, st));
  HE_CUDA_CHECK(cudaStreamSynchronize(st));
  return HE_OK;
}

}  // extern "C"
