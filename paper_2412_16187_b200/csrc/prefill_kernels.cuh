// he_prefill_compress, phases 2 and 3: the sequential replay of Algorithm 1 over the prompt ("Prompt Encoding
// Stage" of Section 3) and the gather of the surviving K / V rows.
//
// Replay: one CTA per (sequence, KV head) unit runs every evicting step t = C..N-1 of that unit in order. The
// unit's code table never leaves the SM: in the main kernel each thread keeps SPT slots in registers, in the
// fallback kernel the table sits in shared memory. Per step: distance of every slot (Eq. 5), packed-key arg-max
// with redux.sync and ONE block barrier (Eq. 6, lowest index on ties), then the slot's own thread rewrites it.
// Warp 0 turns the codes of the next 32 prompt tokens into per-step query contexts one block ahead.
#pragma once
#include "common.cuh"

namespace he {

struct ReplayArgs {
  he_config cfg;
  he_cache ca;
  const uint32_t* kcodes;  // [units, Nmax, Wd]
  const uint32_t* qcodes;  // [units, Nmax, G, Wd]
  const int32_t* prompt_len;
  long long Nmax;
  int smem_slots;  // slots the shared-memory tables were sized for
};

constexpr int kStepBlock = 32;  // prompt tokens whose query contexts are staged at a time (one per lane of warp 0)

// Staging of per-step records [query context | key code] by warp 0, one block of 32 tokens ahead of the scan.
template <int WORDS, int GT>
struct StepStager {
  using Ctx = QueryCtx<WORDS, GT>;
  static constexpr int kRaw = (GT > 0 ? GT : kMaxGroup) * WORDS;
  static constexpr int kRec = Ctx::kRecWords + WORDS;  // words per staged step
  uint32_t rawq[kRaw];
  uint32_t rawk[WORDS];
  bool have;

  __device__ __forceinline__ void prefetch(const uint32_t* qc_u, const uint32_t* kc_u, int t0, int N, int G, int lane) {
    const int t = t0 + lane;
    have = t < N;
    if (have) {
#pragma unroll
      for (int i = 0; i < kRaw; ++i)
        if (i < G * WORDS) rawq[i] = __ldg(qc_u + (long long)t * G * WORDS + i);
#pragma unroll
      for (int w = 0; w < WORDS; ++w) rawk[w] = __ldg(kc_u + (long long)t * WORDS + w);
    }
  }
  __device__ __forceinline__ void commit(uint32_t* stage_buf, int G, int lane) {
    if (have) {
      uint32_t* rec = stage_buf + lane * kRec;
      Ctx::build(rec, rawq, G);
#pragma unroll
      for (int w = 0; w < WORDS; ++w) rec[Ctx::kRecWords + w] = rawk[w];
    }
  }
};

// ------------------------------------------------------------------------------------------------ registers

template <int WORDS, int GT, int SPT, int NT>
__global__ void __launch_bounds__(NT, (NT <= 256 ? 4 : 1)) prefill_replay_reg_kernel(const ReplayArgs a) {
  using Stager = StepStager<WORDS, GT>;
  using Ctx = QueryCtx<WORDS, GT>;
  extern __shared__ __align__(16) int32_t pos_s[];  // [smem_slots]
  __shared__ uint32_t wbest[2][2][32];
  __shared__ uint32_t stage[2][kStepBlock * Stager::kRec];

  const he_config& cfg = a.cfg;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long unit = blockIdx.x;
  const int s = (int)(unit / cfg.n_kv_heads);
  const int G = cfg.group_size;
  const long long Cmax = cfg.max_budget;
  const int C = a.ca.budget[s];
  const int N = a.prompt_len[s];
  const int fill0 = N < C ? N : C;
  const uint32_t* kc_u = a.kcodes + unit * a.Nmax * WORDS;
  const uint32_t* qc_u = a.qcodes + unit * a.Nmax * G * WORDS;
  const bool prot = cfg.n_sink > 0 || cfg.n_recent > 0;
  const bool write_scores = (cfg.flags & HE_FLAG_WRITE_SCORES) != 0;
  float* sc = a.ca.scores + unit * Cmax;

  // the first C tokens fill the cache in order; slot j lives in register j / NT of thread j % NT
  uint32_t code[SPT][WORDS];
#pragma unroll
  for (int r = 0; r < SPT; ++r) {
    const int j = r * NT + tid;
#pragma unroll
    for (int w = 0; w < WORDS; ++w) code[r][w] = j < fill0 ? __ldg(kc_u + (long long)j * WORDS + w) : 0u;
    if (j < fill0) pos_s[j] = j;
  }

  Stager st;
  st.have = false;
  int buf = 0;
  if (C < N && warp == 0) {
    st.prefetch(qc_u, kc_u, C, N, G, lane);
    st.commit(stage[0], G, lane);
  }
  __syncthreads();

  int par = 0;
  for (int t0 = C; t0 < N; t0 += kStepBlock) {
    const bool more = t0 + kStepBlock < N;
    if (more && warp == 0) st.prefetch(qc_u, kc_u, t0 + kStepBlock, N, G, lane);
    const int tend = (N - t0) < kStepBlock ? (N - t0) : kStepBlock;
    for (int ts = 0; ts < tend; ++ts) {
      const int t = t0 + ts;
      const uint32_t* rec = &stage[buf][ts * Stager::kRec];
      Ctx ctx;
      ctx.load(rec, G);
      const bool last = write_scores && (t == N - 1);
      uint32_t best_all = 0u, best_el = 0u;
#pragma unroll
      for (int r = 0; r < SPT; ++r) {
        const int j = r * NT + tid;
        const int rk = ctx.rank(code[r]);
        const uint32_t key = j < C ? (((uint32_t)(rk + 1) << kKeyIdxBits) | (kKeyIdxMask - (uint32_t)j)) : 0u;
        best_all = max(best_all, key);
        if (prot && j < C) {
          const int p = pos_s[j];
          if (p >= cfg.n_sink && p < t - cfg.n_recent) best_el = max(best_el, key);
        }
        if (last && j < C) sc[j] = -(float)ctx.dist(rk);
      }
      uint32_t fin = block_max_key(best_all, wbest[par][0], lane, warp, NT / 32);
      if (prot) {
        best_el = __reduce_max_sync(0xFFFFFFFFu, best_el);
        if (lane == 0) wbest[par][1][warp] = best_el;
        __syncthreads();
        const uint32_t fin_el = __reduce_max_sync(0xFFFFFFFFu, lane < NT / 32 ? wbest[par][1][lane] : 0u);
        if (fin_el != 0u) fin = fin_el;
      }
      const int slot = (int)(kKeyIdxMask - (fin & kKeyIdxMask));
      if (slot % NT == tid) {  // the slot's own scanning thread rewrites it, so no extra barrier is needed
        const int rr = slot / NT;
#pragma unroll
        for (int r = 0; r < SPT; ++r)
          if (r == rr) {
#pragma unroll
            for (int w = 0; w < WORDS; ++w) code[r][w] = rec[Ctx::kRecWords + w];
          }
        pos_s[slot] = t;
      }
      par ^= 1;
    }
    if (more) {
      if (warp == 0) st.commit(stage[buf ^ 1], G, lane);
      __syncthreads();
      buf ^= 1;
    }
  }
  __syncthreads();

  // final state of the unit; everything beyond `fill` is reset
  const bool scored = write_scores && N > C;
#pragma unroll
  for (int r = 0; r < SPT; ++r) {
    const int j = r * NT + tid;
    if (j < Cmax) {
      const bool valid = j < fill0;
#pragma unroll
      for (int w = 0; w < WORDS; ++w) a.ca.codes[(unit * Cmax + j) * WORDS + w] = valid ? code[r][w] : 0u;
      a.ca.pos[unit * Cmax + j] = valid ? pos_s[j] : -1;
      if (!(valid && scored)) sc[j] = 0.f;
    }
  }
  if (tid == 0) {
    a.ca.fill[unit] = fill0;
    a.ca.next_pos[unit] = N;
  }
}

// ------------------------------------------------------------------------------------------------ shared memory

// Fallback for shapes the register kernel is not instantiated for (other group sizes, very large budgets).
template <int WORDS, int GT>
__global__ void prefill_replay_smem_kernel(const ReplayArgs a) {
  using Stager = StepStager<WORDS, GT>;
  using Ctx = QueryCtx<WORDS, GT>;
  extern __shared__ __align__(16) uint32_t rsm[];
  __shared__ uint32_t wbest[2][2][32];
  __shared__ uint32_t stage[2][kStepBlock * Stager::kRec];

  const he_config& cfg = a.cfg;
  const int NT = blockDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = NT >> 5;
  const long long unit = blockIdx.x;
  const int s = (int)(unit / cfg.n_kv_heads);
  const int G = cfg.group_size;
  const long long Cmax = cfg.max_budget;
  const int C = a.ca.budget[s];
  const int N = a.prompt_len[s];
  const int fill0 = N < C ? N : C;
  uint32_t* codes_s = rsm;                                                           // [smem_slots][WORDS]
  int32_t* pos_s = reinterpret_cast<int32_t*>(rsm + (size_t)a.smem_slots * WORDS);  // [smem_slots]
  const uint32_t* kc_u = a.kcodes + unit * a.Nmax * WORDS;
  const uint32_t* qc_u = a.qcodes + unit * a.Nmax * G * WORDS;
  const bool prot = cfg.n_sink > 0 || cfg.n_recent > 0;
  const bool write_scores = (cfg.flags & HE_FLAG_WRITE_SCORES) != 0;
  float* sc = a.ca.scores + unit * Cmax;

  for (int j = tid; j < fill0; j += NT) {
#pragma unroll
    for (int w = 0; w < WORDS; ++w) codes_s[j * WORDS + w] = kc_u[(long long)j * WORDS + w];
    pos_s[j] = j;
  }
  Stager st;
  st.have = false;
  int buf = 0;
  if (C < N && warp == 0) {
    st.prefetch(qc_u, kc_u, C, N, G, lane);
    st.commit(stage[0], G, lane);
  }
  __syncthreads();

  int par = 0;
  for (int t0 = C; t0 < N; t0 += kStepBlock) {
    const bool more = t0 + kStepBlock < N;
    if (more && warp == 0) st.prefetch(qc_u, kc_u, t0 + kStepBlock, N, G, lane);
    const int tend = (N - t0) < kStepBlock ? (N - t0) : kStepBlock;
    for (int ts = 0; ts < tend; ++ts) {
      const int t = t0 + ts;
      const uint32_t* rec = &stage[buf][ts * Stager::kRec];
      Ctx ctx;
      ctx.load(rec, G);
      const bool last = write_scores && (t == N - 1);
      uint32_t best_all = 0u, best_el = 0u;
      for (int j = tid; j < C; j += NT) {
        uint32_t h[WORDS];
#pragma unroll
        for (int w = 0; w < WORDS; ++w) h[w] = codes_s[j * WORDS + w];
        const int rk = ctx.rank(h);
        const uint32_t key = ((uint32_t)(rk + 1) << kKeyIdxBits) | (kKeyIdxMask - (uint32_t)j);
        best_all = max(best_all, key);
        if (prot) {
          const int p = pos_s[j];
          if (p >= cfg.n_sink && p < t - cfg.n_recent) best_el = max(best_el, key);
        }
        if (last) sc[j] = -(float)ctx.dist(rk);
      }
      uint32_t fin = block_max_key(best_all, wbest[par][0], lane, warp, nwarps);
      if (prot) {
        best_el = __reduce_max_sync(0xFFFFFFFFu, best_el);
        if (lane == 0) wbest[par][1][warp] = best_el;
        __syncthreads();
        const uint32_t fin_el = __reduce_max_sync(0xFFFFFFFFu, lane < nwarps ? wbest[par][1][lane] : 0u);
        if (fin_el != 0u) fin = fin_el;
      }
      const int slot = (int)(kKeyIdxMask - (fin & kKeyIdxMask));
      if (slot % NT == tid) {
#pragma unroll
        for (int w = 0; w < WORDS; ++w) codes_s[slot * WORDS + w] = rec[Ctx::kRecWords + w];
        pos_s[slot] = t;
      }
      par ^= 1;
    }
    if (more) {
      if (warp == 0) st.commit(stage[buf ^ 1], G, lane);
      __syncthreads();
      buf ^= 1;
    }
  }
  __syncthreads();

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

// ------------------------------------------------------------------------------------------------ gather

struct GatherArgs {
  he_config cfg;
  he_cache ca;
  const void* k;
  const void* v;
  long long s0, s1, s2;
};

constexpr int kGatherThreads = 256;
constexpr int kGatherUnroll = 4;

// K[unit, j] = k[s, h, pos[j]] and the same for V: 16 bytes per thread, four loads in flight per thread.
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

}  // namespace he
