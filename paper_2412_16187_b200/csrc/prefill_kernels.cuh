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
  int32_t* sched;  // unit schedule written by prefill_schedule_kernel
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

// ------------------------------------------------------------------------------------------------ scheduling

// Replay work is very uneven when budgets are ragged (a unit costs about (N - C) * C slot visits) and a CTA
// runs one unit at a time, so units are sorted by work and dealt to one bin per SM, largest first, in a snake over
// the bins. A replay CTA drains the bin of the SM it runs on and then helps other bins. The result never depends on
// which CTA runs which unit; only the time does.
//
// sched layout (int32): [0] nbins, [1] units, [2 .. 2+nbins] bin_start (nbins + 1 entries),
//                       [3+nbins .. 3+2*nbins) cursor, then order[units] (unit ids grouped by bin).
constexpr int kMaxBins = 256;
constexpr int kSchedSortMax = 4096;  // more units than this are dealt round-robin (they balance by number)
constexpr int kSchedThreads = 1024;

__host__ __device__ inline size_t sched_words(long long units) { return 3 + 2 * (size_t)kMaxBins + (size_t)units; }

// step_cost: fixed cost of one evicting step in units of one slot scanned (0 for the register kernel, whose step is a
// scan; several thousand for the tensor-core kernel, whose step is mostly the resolver's latency).
__global__ void __launch_bounds__(kSchedThreads) prefill_schedule_kernel(const he_config cfg, const int32_t* budget,
                                                                          const int32_t* prompt_len, int nbins,
                                                                          int32_t* sched, int step_cost) {
  __shared__ unsigned long long keys[kSchedSortMax];  // (work << 20) | (0xFFFFF - unit), sorted descending
  __shared__ int start_s[kMaxBins];
  __shared__ unsigned char bin_of[kSchedSortMax];  // nbins <= 256
  __shared__ unsigned short pos_of[kSchedSortMax];  // place of the unit inside its bin
  const int tid = threadIdx.x;
  const int units = cfg.batch * cfg.n_kv_heads;
  int32_t* bin_start = sched + 2;
  int32_t* cursor = sched + 3 + nbins;
  int32_t* order = sched + 3 + 2 * nbins;
  if (tid == 0) {
    sched[0] = nbins;
    sched[1] = units;
  }
  for (int i = tid; i < nbins; i += kSchedThreads) cursor[i] = 0;
  if (units > kSchedSortMax) {  // plenty of units: round-robin bins
    for (int b = tid; b <= nbins; b += kSchedThreads) {
      // bin b holds units b, b + nbins, ...: count = ceil((units - b) / nbins)
      long long before = 0;
      for (int k = 0; k < b; ++k) before += (units - k + nbins - 1) / nbins;
      bin_start[b] = (int)before;
    }
    for (int u = tid; u < units; u += kSchedThreads) {
      const int b = u % nbins;
      long long before = 0;
      for (int k = 0; k < b; ++k) before += (units - k + nbins - 1) / nbins;
      order[before + u / nbins] = u;
    }
    return;
  }
  int n = 1;
  while (n < units) n <<= 1;
  for (int i = tid; i < n; i += kSchedThreads) {
    unsigned long long key = 0ull;
    if (i < units) {
      const int s = i / cfg.n_kv_heads;
      const long long C = clamp_budget(budget[s], cfg.max_budget), N = clamp_len(prompt_len[s], 0x7FFFFFFF, (int)C);
      const long long work = N > C ? (N - C) * (C + step_cost) + 1 : 1;  // evicting steps x (slots scanned + fixed cost)
      key = ((unsigned long long)work << 20) | (unsigned long long)(0xFFFFF - i);
    }
    keys[i] = key;
  }
  __syncthreads();
  for (int k = 2; k <= n; k <<= 1)  // bitonic sort, descending
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int i = tid; i < n; i += kSchedThreads) {
        const int l = i ^ j;
        if (l > i) {
          const unsigned long long a = keys[i], b = keys[l];
          const bool desc = (i & k) == 0;
          if (desc ? a < b : a > b) {
            keys[i] = b;
            keys[l] = a;
          }
        }
      }
      __syncthreads();
    }
  // Sorted units are dealt to the bins in a snake (ranks 0 .. nbins-1 forwards, the next nbins backwards, ...): every
  // bin gets one unit of each round, the heavy bins of one round the light units of the next. A greedy
  // lightest-bin-first deal balances a little better on paper but is a serial loop over the units (65 us for 512 of
  // them, 2 % of the call), and the replay CTAs steal from other bins once their own is empty, which evens out what
  // the deal leaves (measured: the call time does not depend on the cost model at all).
  const int rounds_full = units / nbins, rem = units - rounds_full * nbins;
  for (int bb = tid; bb <= nbins; bb += kSchedThreads) {
    // units in bins below bb: the full rounds give each bin one; the partial round (if any) fills from the front when
    // its number is even and from the back when it is odd
    const int extra = (rounds_full & 1) == 0 ? min(bb, rem) : max(0, bb - (nbins - rem));
    const int st = bb * rounds_full + extra;
    if (bb < nbins) start_s[bb] = st;
    bin_start[bb] = st;
  }
  for (int i = tid; i < units; i += kSchedThreads) {
    const int round = i / nbins, k = i - round * nbins;
    bin_of[i] = (unsigned char)((round & 1) == 0 ? k : nbins - 1 - k);
    pos_of[i] = (unsigned short)round;
  }
  __syncthreads();
  // sorted order, so each bin lists its largest unit first
  for (int i = tid; i < units; i += kSchedThreads) order[start_s[bin_of[i]] + pos_of[i]] = 0xFFFFF - (int)(keys[i] & 0xFFFFF);
}

// Next unit for this CTA: from the bin of the SM it runs on, else from the first other bin that still has work.
// Returns -1 when every bin is drained. Called by warp 0; every unit is handed out exactly once.
__device__ __forceinline__ int claim_unit(int32_t* sched, int lane) {
  const int nbins = sched[0];
  const int32_t* bin_start = sched + 2;
  int32_t* cursor = sched + 3 + nbins;
  const int32_t* order = sched + 3 + 2 * nbins;
  unsigned smid;
  asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
  const int home = (int)(smid % (unsigned)nbins);
  for (int base = 0; base < nbins; base += 32) {
    const int b = (home + base + lane) % nbins;
    const bool in_range = base + lane < nbins;
    const int cnt = in_range ? bin_start[b + 1] - bin_start[b] : 0;
    bool avail = in_range && *reinterpret_cast<volatile int32_t*>(cursor + b) < cnt;
    unsigned m = __ballot_sync(0xFFFFFFFFu, avail);
    while (m) {
      const int src = __ffs(m) - 1;
      int got = -1;
      if (lane == src) {
        const int idx = atomicAdd(cursor + b, 1);
        if (idx < cnt) got = order[bin_start[b] + idx];
      }
      got = __shfl_sync(0xFFFFFFFFu, got, src);
      if (got >= 0) return got;
      m &= m - 1;  // that bin was drained in the meantime
    }
  }
  return -1;
}

// ------------------------------------------------------------------------------------------------ registers

template <int WORDS, int GT, int SPT, int NT>
__global__ void __launch_bounds__(NT, (NT <= 256 ? 4 : (NT <= 512 ? 2 : 1))) prefill_replay_reg_kernel(const ReplayArgs a) {
  using Stager = StepStager<WORDS, GT>;
  using Ctx = QueryCtx<WORDS, GT>;
  extern __shared__ __align__(16) int32_t pos_s[];  // [smem_slots]
  __shared__ uint32_t wbest[2][2][32];
  __shared__ uint32_t stage[2][kStepBlock * Stager::kRec];
  __shared__ int s_unit;
  static_assert(SPT <= 32, "the per-thread key packs the register index in 5 bits");

  const he_config& cfg = a.cfg;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = cfg.group_size;
  const long long Cmax = cfg.max_budget;
  const bool prot = cfg.n_sink > 0 || cfg.n_recent > 0;
  const bool write_scores = (cfg.flags & HE_FLAG_WRITE_SCORES) != 0;

  for (;;) {
    if (warp == 0) {
      const int u = claim_unit(a.sched, lane);
      if (lane == 0) s_unit = u;
    }
    __syncthreads();
    const long long unit = s_unit;
    if (unit < 0) break;
    const int s = (int)(unit / cfg.n_kv_heads);
    const int C = clamp_budget(a.ca.budget[s], (int)Cmax);
    const int N = clamp_len(a.prompt_len[s], a.Nmax, C);
    const int fill0 = N < C ? N : C;
    const uint32_t* kc_u = a.kcodes + unit * a.Nmax * WORDS;
    const uint32_t* qc_u = a.qcodes + unit * a.Nmax * G * WORDS;
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
    const int nfull = C / NT;             // registers that hold a valid slot in every thread
    const bool has_tail = tid < C % NT;   // register nfull holds a valid slot in the first C % NT threads
    const int nregs = (C + NT - 1) / NT;  // registers that hold a valid slot in some thread
    const uint32_t vmask = (nfull >= 32 ? 0xFFFFFFFFu : ((1u << nfull) - 1u)) | (has_tail ? (1u << nfull) : 0u);  // bit r: slot valid

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
        // thread-local arg-max over its registers: key = rank * 32 + (31 - r), so equal ranks keep the lower slot.
        // Registers are visited in groups of four. The common step (no protected window, not the scoring step)
        // is branch-free inside a group; only the group that straddles the budget masks invalid slots.
        int loc_all = -1, loc_el = -1;
        if (!prot && !last) {
#pragma unroll
          for (int g0 = 0; g0 < SPT; g0 += 4) {
            if (g0 >= nregs) break;  // uniform over the block
            if (g0 + 4 <= nfull) {
#pragma unroll
              for (int r = g0; r < g0 + 4 && r < SPT; ++r) loc_all = max(loc_all, ctx.rank(code[r]) * 32 + (31 - r));
            } else {
#pragma unroll
              for (int r = g0; r < g0 + 4 && r < SPT; ++r) {
                const int key = ctx.rank(code[r]) * 32 + (31 - r);
                loc_all = max(loc_all, ((vmask >> r) & 1u) ? key : -1);
              }
            }
          }
        } else {
#pragma unroll
          for (int r = 0; r < SPT; ++r) {
            if ((vmask >> r) & 1u) {
              const int rk = ctx.rank(code[r]);
              const int key = rk * 32 + (31 - r);
              loc_all = max(loc_all, key);
              if (prot) {
                const int p = pos_s[r * NT + tid];
                if (p >= cfg.n_sink && p < t - cfg.n_recent) loc_el = max(loc_el, key);
              }
              if (last) sc[r * NT + tid] = -(float)ctx.dist(rk);
            }
          }
        }
        // block-wide key = (rank + 1) << 20 | (0xFFFFF - slot); 0 when the thread has no (eligible) slot
        auto widen = [&](int loc) -> uint32_t {
          if (loc < 0) return 0u;
          const int r = 31 - (loc & 31);
          return ((uint32_t)((loc >> 5) + 1) << kKeyIdxBits) | (kKeyIdxMask - (uint32_t)(r * NT + tid));
        };
        uint32_t fin = block_max_key(widen(loc_all), wbest[par][0], lane, warp, NT / 32);
        if (prot) {
          uint32_t best_el = __reduce_max_sync(0xFFFFFFFFu, widen(loc_el));
          if (lane == 0) wbest[par][1][warp] = best_el;
          __syncthreads();
          const uint32_t fin_el = __reduce_max_sync(0xFFFFFFFFu, lane < NT / 32 ? wbest[par][1][lane] : 0u);
          if (fin_el != 0u) fin = fin_el;
        }
        const int slot = (int)(kKeyIdxMask - (fin & kKeyIdxMask));
        if (slot % NT == tid && HE_IN_RANGE(slot, C)) {  // the slot's own scanning thread rewrites it, so no extra barrier is needed
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
        uint32_t cw[WORDS];
#pragma unroll
        for (int w = 0; w < WORDS; ++w) cw[w] = valid ? code[r][w] : 0u;
        store_slot_code<WORDS>(a.cfg, a.ca.codes, unit * Cmax + j, cw);
        a.ca.pos[unit * Cmax + j] = valid ? pos_s[j] : -1;
        if (!(valid && scored)) sc[j] = 0.f;
      }
    }
    if (tid == 0) {
      a.ca.fill[unit] = fill0;
      a.ca.next_pos[unit] = N;
    }
    __syncthreads();  // pos_s, stage and s_unit are reused by the next unit
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
  const int C = clamp_budget(a.ca.budget[s], (int)Cmax);
  const int N = clamp_len(a.prompt_len[s], a.Nmax, C);
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
      if (slot % NT == tid && HE_IN_RANGE(slot, C)) {
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
    uint32_t cw[WORDS];
#pragma unroll
    for (int w = 0; w < WORDS; ++w) cw[w] = valid ? codes_s[j * WORDS + w] : 0u;
    store_slot_code<WORDS>(a.cfg, a.ca.codes, unit * Cmax + j, cw);
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
  long long Nmax;  // prompt tokens per unit in k, v
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
  const int fill = min(max(a.ca.fill[unit], 0), (int)Cmax);
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
      if (!HE_IN_RANGE(tok, a.Nmax)) continue;  // (a slot of a valid cache names a prompt token)
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

// The same copy for rows of a power-of-two number of 16-byte chunks (every supported head size but the odd ones): a
// group of `cpr` threads owns a slot at a time, reads its position once and moves the K row and the V row, 16 bytes each
// per thread; kGatherRows slots per group, so eight loads per thread are in flight. No division anywhere.
constexpr int kGatherRows = 4;
__global__ void __launch_bounds__(kGatherThreads) prefill_gather_rows_kernel(const GatherArgs a, int lg_cpr) {
  const he_config& cfg = a.cfg;
  const long long unit = blockIdx.y;
  const int s = (int)(unit / cfg.n_kv_heads), h = (int)(unit % cfg.n_kv_heads);
  const int es = esize_of(cfg.dtype);
  const long long Cmax = cfg.max_budget;
  const int fill = min(max(a.ca.fill[unit], 0), (int)Cmax);
  const int groups = kGatherThreads >> lg_cpr;
  const int j0 = blockIdx.x * groups * kGatherRows;
  if (j0 >= fill) return;
  const int ch = threadIdx.x & ((1 << lg_cpr) - 1), g = threadIdx.x >> lg_cpr;
  const int32_t* pp = a.ca.pos + unit * Cmax;
  const char* kb = static_cast<const char*>(a.k) + (s * a.s0 + h * a.s1) * es;
  const char* vb = static_cast<const char*>(a.v) + (s * a.s0 + h * a.s1) * es;
  long long tok[kGatherRows];
#pragma unroll
  for (int i = 0; i < kGatherRows; ++i) {
    const int j = j0 + i * groups + g;
    tok[i] = -1;
    if (j < fill) {
      const long long tk = __ldg(pp + j);
      if (HE_IN_RANGE(tk, a.Nmax)) tok[i] = tk;  // (a slot of a valid cache names a prompt token)
    }
  }
  uint4 kv[kGatherRows], vv[kGatherRows];
#pragma unroll
  for (int i = 0; i < kGatherRows; ++i)
    if (tok[i] >= 0) {
      kv[i] = __ldg(reinterpret_cast<const uint4*>(kb + tok[i] * a.s2 * es) + ch);
      vv[i] = __ldg(reinterpret_cast<const uint4*>(vb + tok[i] * a.s2 * es) + ch);
    }
  uint4* kd = reinterpret_cast<uint4*>(a.ca.k_cache) + ((unit * Cmax) << lg_cpr) + ch;
  uint4* vd = reinterpret_cast<uint4*>(a.ca.v_cache) + ((unit * Cmax) << lg_cpr) + ch;
#pragma unroll
  for (int i = 0; i < kGatherRows; ++i)
    if (tok[i] >= 0) {
      const long long j = j0 + i * groups + g;
      kd[j << lg_cpr] = kv[i];
      vd[j << lg_cpr] = vv[i];
    }
}

}  // namespace he
