// he_prefill_compress, phase 2 on the tensor cores: the sequential replay of Algorithm 1 over the prompt ("Prompt
// Encoding Stage" of Section 3) with the Hamming distances of Eq. 5 taken 128 steps at a time as a dense product.
//
// Why this is a contraction. With codes read as +-1 vectors s, the group distance of slot j at step t is
//   D(j, t) = sum_g popc(h_j xor h(q_{t,g})) = (G * K - <s_j, u_t>) / 2,   u_t = sum_g s(q_{t,g})  (entries in -G..G),
// so the distances of all slots to a block of steps are one [steps x K] * [K x slots] product of small integers,
// exact in bf16 operands and fp32 accumulation. Three more columns of the contraction turn the accumulator into
// the arg-max key of Eq. 6 itself:  key(j, t) = D * 2^14 + (16383 - j)  (largest distance first, lowest slot on
// ties): A = [-2^13 u_t | 128 | 1 | G K 2^13], B = [s_j | idx_j >> 7 | idx_j & 127 | 1], idx_j = 16383 - j. Every
// partial sum is an integer below 2^24, so the result does not depend on the order of accumulation.
//
// What stays sequential. Step t must see the table as steps < t left it. A block of 128 steps is multiplied
// against the table as it stood at the start of the block ("base" slots), and one more tile holds the distances
// of the block's own 128 keys to the block's queries ("new" entries). A single warp then walks the block's steps
// in order: the step's best base slot comes from per-tile maxima that the tensor-memory readers left in shared
// memory, its best new entry from the extra tile, and a slot that an earlier step of the block has already evicted
// is recognised by an owner table; only then is that tile's maximum recomputed for this step with popcounts. If
// a block meets many such repairs it is cut short and the next block starts from the updated table, which bounds
// the cost on adversarial data. The result is bit for bit that of the step-by-step scan.
//
// One persistent CTA per SM (units claimed from the same schedule as the register kernel), 416 threads:
//   warps 0-3  read accumulators from tensor memory (one step per thread), reduce each 128-slot tile to its maximum
//              key; warp 0 is also the resolver that walks the steps of a block
//   warps 4-11 expand packed codes into +-1 bf16 operand tiles (K-major, 128-byte swizzle), one slot per thread,
//              four warps per operand stage
//   warp 12    one thread issues the tcgen05.mma instructions (M = 128 steps, N = 128 slots, K = 16) and commits
// Every wait on an mbarrier is bounded; on a time-out the CTA raises a flag, leaves its loops through the same
// barriers as usual, releases tensor memory and returns, and the device error counter is incremented.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "hash_tc_kernels.cuh"
#include "prefill_kernels.cuh"

namespace he {

constexpr int kRtThreads = 416;
constexpr int kRtMmaWarp = kRtThreads / 32 - 1;
constexpr int kRtRows = 128;       // steps per block = MMA M
constexpr int kRtTile = 128;       // slots per tile = MMA N
constexpr int kRtMaxSlots = 4096;         // largest budget whose code and position tables stay in shared memory
constexpr int kRtMaxSlotsGlobal = 12288;  // largest budget at all: the tables then live in the cache's own arrays
constexpr int kRtKeyShift = 14;
constexpr int kRtIdxMask = (1 << kRtKeyShift) - 1;
constexpr int kRtStaleLimit = 64;  // repairs after which a block is cut short
constexpr int kRtSecondMaxTiles = 8;  // tables up to this many tiles also keep each tile's second-largest key (8-bit operands)
constexpr int kRtFastNum = 3, kRtFastDen = 10;  // run-based resolver while fewer than NUM / DEN of a unit's steps are not easy
constexpr int kRtAtomBytes = kRtRows * 128;  // one 64-column K-major swizzle atom of a 128-row operand tile

__device__ __forceinline__ void tc_mma_f8(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"((uint32_t)accumulate)
      : "memory");
}

// e4m3 bit pattern of a small non-negative integer with at most four significant bits (exact).
__device__ __forceinline__ uint32_t rt_e4m3_of_int(int v) {
  if (v <= 0) return 0u;
  const int p = 31 - __clz(v);
  const uint32_t mant = p >= 3 ? ((uint32_t)v >> (p - 3)) & 7u : ((uint32_t)v << (3 - p)) & 7u;
  return ((uint32_t)(p + 7) << 3) | mant;
}

// Byte offsets of the kernel's dynamic shared memory (after rounding its base up to 1024 bytes).
struct RtLayout {
  uint32_t a, b, codes, pos, owner, m, m2, rb, ub, ps, es, dn, qraw, kraw, total;
};
// `slots` is the budget rounded up to whole tiles; the tile-maximum table has an odd pitch (conflict-free column writes).
__host__ __device__ inline int rt_mpitch(int slots, bool table_in_smem) { return table_in_smem ? kRtMaxSlots / kRtTile + 1 : ((slots / kRtTile) | 1); }
__host__ __device__ inline RtLayout rt_layout(int words, int slots, int G, bool table_in_smem, bool fp8) {
  RtLayout L;
  const uint32_t atoms = (words == 2 && !fp8) ? 2u : 1u;  // 8-bit operands: a row of codes and key columns fits 128 bytes
  const uint32_t stages = fp8 ? 4u : 2u;
  uint32_t o = 0;
  L.a = o, o += atoms * kRtAtomBytes;
  L.b = o, o += stages * atoms * kRtAtomBytes;
  L.codes = o, o += table_in_smem ? (uint32_t)slots * words * 4u : 0u;
  L.pos = o, o += table_in_smem ? (uint32_t)slots * 4u : 0u;
  L.owner = o, o += (uint32_t)slots * 2u;
  L.m = o, o += (uint32_t)kRtRows * rt_mpitch(slots, table_in_smem) * 4u;
  // second-largest key per (step, tile): kept where it fits (tables in shared memory, 8-bit operands)
  L.m2 = o, o += (table_in_smem && fp8) ? (uint32_t)kRtRows * rt_mpitch(slots, true) * 4u : 0u;
  L.rb = o, o += kRtRows * 4u;
  L.ub = o, o += kRtRows * 4u;
  L.ps = o, o += kRtRows * 4u;
  L.es = o, o += kRtRows * 4u;
  L.dn = o, o += kRtRows * kRtRows * 2u;
  L.qraw = o, o += 2u * kRtRows * G * words * 4u;  // two buffers: this block's codes and the next block's
  L.kraw = o, o += 2u * kRtRows * words * 4u;
  L.total = o + 1024u;
  return L;
}

// Byte offset of 16-byte chunk `chunk` (0..7) of row `row` inside one swizzle atom.
__device__ __forceinline__ uint32_t rt_swz(int row, int chunk) {
  return (uint32_t)((row >> 3) * 1024 + (row & 7) * 128 + ((chunk ^ (row & 7)) << 4));
}

// bf16 bit pattern of a small non-negative integer (< 256: exact).
__device__ __forceinline__ uint32_t rt_bf16_of_int(int x) { return __float_as_uint((float)x) >> 16; }

// Eight code bits (bits 8c .. 8c+7 of the code) as eight +-1 bf16 values: bit set -> +1 (0x3F80), clear -> -1 (0xBF80).
__device__ __forceinline__ uint4 rt_expand8(uint32_t byte) {
  const uint32_t x = ~byte;
  uint4 v;
  v.x = 0x3F803F80u | ((x << 15) & 0x8000u) | ((x << 30) & 0x80000000u);
  v.y = 0x3F803F80u | ((x << 13) & 0x8000u) | ((x << 28) & 0x80000000u);
  v.z = 0x3F803F80u | ((x << 11) & 0x8000u) | ((x << 26) & 0x80000000u);
  v.w = 0x3F803F80u | ((x << 9) & 0x8000u) | ((x << 24) & 0x80000000u);
  return v;
}

// Largest of three floats in one instruction (sm_100 has the three-input form).
__device__ __forceinline__ float rt_fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Group distance of Eq. 5 straight from the packed words (used for the few slots the resolver looks at itself).
template <int WORDS>
__device__ __forceinline__ int rt_dist(const uint32_t* h, const uint32_t* q, int G) {
  int D = 0;
  for (int g = 0; g < G; ++g) {
#pragma unroll
    for (int w = 0; w < WORDS; ++w) D += __popc(h[w] ^ q[g * WORDS + w]);
  }
  return D;
}

// GLOBAL_TABLE: the unit's code and position tables are the cache's own arrays in global memory (budgets beyond
// kRtMaxSlots); otherwise they sit in shared memory and are written out when the unit is done.
// 13 warps: one scheduler hosts four of them, so 128 registers per thread is the most its 16 K registers allow.
// FP8 (group sizes up to 7): operand A in e5m2 (-2^13 u_t with |u_t| <= 7 is exact), operand B in e4m3 (+-1 and
// the digits of the slot index), K = 32 per instruction: half the operand bytes and three instructions per tile
// instead of five, four operand stages and four accumulators. The key columns are then
//   A = [.. | 2^14 | 4096 | 256 | 16 | 1],  B = [.. | G K / 2 | idx >> 12 | (idx >> 8) & 15 | (idx >> 4) & 15 | idx & 15].
// PROT (protected windows, Section 4 setup: the first n_sink prompt tokens and the n_recent newest tokens are never
// evicted; requires every budget > n_sink + n_recent so that some slot is always eligible): nothing changes in the
// operands. The resolver treats a best base slot that is not eligible at this step like a stale one (the repair
// then takes the tile's best eligible slot), and a token that enters at step r joins the new entries only at step
// r + n_recent + 1, when it stops being recent; until then, and in the next block, it cannot win.
// RUNS = false leaves the run-based resolver loop out of the kernel: for launches none of whose units can use it (see
// `second` below) the sequential loop alone compiles to tighter code (5 % of the call at 1024-slot budgets).
template <int WORDS, bool GLOBAL_TABLE, bool FP8, bool PROT = false, bool RUNS = true>
__global__ void __launch_bounds__(kRtThreads, 1) prefill_replay_tc_kernel(const ReplayArgs a) {
  constexpr bool kRuns = RUNS && !PROT;
  constexpr int ATOMS = (WORDS == 2 && !FP8) ? 2 : 1;
  constexpr int KB = 32 * WORDS;             // code columns of the contraction
  constexpr int KSTEPS = FP8 ? KB / 32 + 1 : (KB + 16) / 16;  // MMA instructions per tile (the last one holds the key columns)
  constexpr int ESZ = FP8 ? 1 : 2;           // bytes per operand element
  constexpr int XATOM = (KB * ESZ) / 128, XCHUNK = ((KB * ESZ) % 128) / 16;  // where the key columns start
  constexpr int NSTAGE = FP8 ? 4 : 2;        // operand stages = accumulators in tensor memory
  // Tiles per hand-over: with four stages two consecutive tiles (one per expander group) travel together, so every
  // role waits on its mbarriers once per 256 slots instead of once per 128 (a wait costs about as much as a quarter
  // of a tile's work even when the barrier is already complete).
  constexpr int TP = FP8 ? 2 : 1;
  constexpr int NSYNC = NSTAGE / TP;         // hand-over slots: stage pair (or stage) + accumulator pair (or accumulator)
  constexpr int NT = kRtThreads;
  extern __shared__ unsigned char rt_smem_raw[];
  __shared__ __align__(8) unsigned long long bars[4 * NSTAGE + 1];  // the last one: drain barrier of the abort path
  __shared__ uint32_t tmem_base_s;
  __shared__ volatile int abort_flag;
  __shared__ int s_unit, s_done, s_fast, s_hold, s_backoff;
  __shared__ uint16_t entry_slot[PROT ? kRtRows : 1];  // PROT: the slot each of the block's steps wrote to
  // four code bits -> four bf16 values: operand B takes +-1 (bit set: +1), operand A -+2^13 (bit set: -2^13)
  __shared__ uint2 s_lut_a[16], s_lut_b[16];
  // 8-bit operands: operand A is summed in f16 (-+2^13 per head) and keeps the high bytes (= e5m2); operand B takes a
  // whole code byte -> eight e4m3 values of +-1
  __shared__ uint2 s_lut_b8[FP8 ? 256 : 1];

  const he_config& cfg = a.cfg;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = cfg.group_size;
  const long long Cmax = cfg.max_budget;
  const bool write_scores = (cfg.flags & HE_FLAG_WRITE_SCORES) != 0;
  // rounded up to 1024 bytes by an offset from the array itself, so that the compiler still knows these are
  // shared-memory addresses (a round trip through an integer would turn every access into a generic one)
  unsigned char* smem = rt_smem_raw + ((1024u - (smem_u32(rt_smem_raw) & 1023u)) & 1023u);
  const RtLayout L = rt_layout(WORDS, a.smem_slots, G, !GLOBAL_TABLE, FP8);
  const int mp = GLOBAL_TABLE ? rt_mpitch(a.smem_slots, false) : kRtMaxSlots / kRtTile + 1;  // a constant for the smaller tables
  unsigned char* As = smem + L.a;
  unsigned char* Bs = smem + L.b;
  int16_t* owner = reinterpret_cast<int16_t*>(smem + L.owner);
  int32_t* Mx = reinterpret_cast<int32_t*>(smem + L.m);
  // The readers may also keep each tile's second-largest key. Not in the kernel that holds the run-based loop: there the
  // leaner code is worth more than the repairs those keys save (3.00 against 3.08 ms per call on ragged 512..4096 budgets).
  constexpr bool SECOND = FP8 && !GLOBAL_TABLE && !kRuns;
  int32_t* Mx2 = reinterpret_cast<int32_t*>(smem + L.m2);
  int32_t* RB = reinterpret_cast<int32_t*>(smem + L.rb);
  int32_t* UB = reinterpret_cast<int32_t*>(smem + L.ub);  // per step: no new entry's key can exceed this
  int32_t* PS = reinterpret_cast<int32_t*>(smem + L.ps);  // per step: slot of the best base key, flags (see the readers)
  int32_t* ES = reinterpret_cast<int32_t*>(smem + L.es);  // per new entry of the block: 16383 - its slot while resident
  uint16_t* Dn = reinterpret_cast<uint16_t*>(smem + L.dn);
  uint32_t* qraw = reinterpret_cast<uint32_t*>(smem + L.qraw);
  uint32_t* kraw = reinterpret_cast<uint32_t*>(smem + L.kraw);

  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };          // expanders -> MMA: operand stage s is written
  auto tfull_bar = [&](int x) { return bar0 + 8u * (2 * NSTAGE + x); };   // MMA -> readers: accumulator x is complete
  auto empty_bar = tfull_bar;                                              // MMA -> expanders: stage x has been read (same event)
  auto tempty_bar = [&](int x) { return bar0 + 8u * (3 * NSTAGE + x); };  // readers -> MMA: accumulator x is drained
  if (tid == 0) {
    abort_flag = 0;
    mbar_init(bar0 + 8u * (4 * NSTAGE), 1);
    for (int s = 0; s < NSTAGE; ++s) {
      mbar_init(full_bar(s), 4 * TP);  // one arrival per expander warp
      mbar_init(tfull_bar(s), 1);
      mbar_init(tempty_bar(s), 4);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < 16) {
    auto pick = [&](int bit, uint32_t set, uint32_t clear) { return ((tid >> bit) & 1) ? set : clear; };
    s_lut_b[tid] = make_uint2(pick(0, 0x3F80u, 0xBF80u) | (pick(1, 0x3F80u, 0xBF80u) << 16),
                              pick(2, 0x3F80u, 0xBF80u) | (pick(3, 0x3F80u, 0xBF80u) << 16));
    const uint32_t a_set = FP8 ? 0xF000u : 0xC600u, a_clr = FP8 ? 0x7000u : 0x4600u;  // -+2^13 as f16 / bf16
    s_lut_a[tid] = make_uint2(pick(0, a_set, a_clr) | (pick(1, a_set, a_clr) << 16), pick(2, a_set, a_clr) | (pick(3, a_set, a_clr) << 16));
  }
  if (FP8 && tid < 256) {
    uint32_t lo = 0u, hi = 0u;
    for (int k = 0; k < 4; ++k) {
      lo |= (((tid >> k) & 1) ? 0x38u : 0xB8u) << (8 * k);
      hi |= (((tid >> (k + 4)) & 1) ? 0x38u : 0xB8u) << (8 * k);
    }
    s_lut_b8[tid] = make_uint2(lo, hi);
  }
  if (warp == kRtMmaWarp) {  // NSTAGE accumulators of 128 columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(NSTAGE * kRtTile)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  // instruction descriptor: fp32 accumulate; operand formats bf16 x bf16 (kind::f16: 1, 1) or e5m2 x e4m3
  // (kind::f8f6f4: 1, 0); both operands K-major; N = 128, M = 128
  const uint32_t idesc = (1u << 4) | (1u << 7) | ((FP8 ? 0u : 1u) << 10) | ((uint32_t)(kRtTile >> 3) << 17) |
                         ((uint32_t)(kRtRows >> 4) << 24);
  const uint32_t kconst_bits = __float_as_uint((float)(G * KB / 2) * 16384.f) >> 16;  // exact: G K / 2 <= 256
  const uint32_t cst_e4m3 = rt_e4m3_of_int(G * KB / 2);
  int it = 0;  // hand-overs (groups of TP tiles) so far; every role counts the same sequence

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
    const int nbase = (C + kRtTile - 1) / kRtTile;
    // The second-largest key per (step, tile) lets most stale maxima be settled without recomputing a tile, but costs
    // the readers five instructions per two elements instead of one. Measured on B200: with 1024 slots (8 tiles, a
    // fifth of the steps stale) the call gets 8 % faster, with 2048 slots and more the longer tile phase costs more
    // than the repairs saved.
    const bool second = SECOND && nbase <= kRtSecondMaxTiles;
    uint32_t* codes_t = GLOBAL_TABLE ? a.ca.codes + unit * Cmax * WORDS : reinterpret_cast<uint32_t*>(smem + L.codes);
    int32_t* pos_t = GLOBAL_TABLE ? a.ca.pos + unit * Cmax : reinterpret_cast<int32_t*>(smem + L.pos);
    // the first C tokens fill the cache in order; everything beyond `fill` is reset
    for (int j = tid; j < (GLOBAL_TABLE ? (int)Cmax : a.smem_slots); j += NT) {
#pragma unroll
      for (int w = 0; w < WORDS; ++w) codes_t[j * WORDS + w] = j < fill0 ? __ldg(kc_u + (long long)j * WORDS + w) : 0u;
      pos_t[j] = j < fill0 ? j : -1;
    }
    // PROT with the tables in global memory: positions are too far away for the resolver's step-ahead checks, so warp 0
    // keeps the slots of the 32 newest tokens in a register ring (lane l: the newest token congruent to l mod 32; the
    // first C tokens sit in slot = position) and sinks are recognised by their slot (they never leave slots 0..n_sink-1).
    if (tid == 0) {
      s_fast = 0;  // a unit's first block runs the sequential loop and counts
      s_hold = 0;
      s_backoff = 2;
    }
    int myring = -1;
    if (PROT && GLOBAL_TABLE) {
      const int pl = fill0 - 1 - ((fill0 - 1 - lane) & 31);
      myring = pl >= 0 ? pl : -1;
    }
    // A table word as the latest step left it (global tables: read past L1, which other warps' stores do not update)
    auto table_word = [&](int idx) -> uint32_t { return GLOBAL_TABLE ? __ldcg(codes_t + idx) : codes_t[idx]; };
    auto table_pos = [&](int j) -> int { return GLOBAL_TABLE ? __ldcg(pos_t + j) : pos_t[j]; };
    __syncthreads();
    bool aborted = false;
    const int GW = G * WORDS;
    // The block's query and key codes into buffer `buf` (rows past the prompt are zero).
    auto stage_codes = [&](int buf, int tb, int nrows, int first, int nthreads) {
      uint32_t* qd = qraw + buf * kRtRows * GW;
      uint32_t* kd = kraw + buf * kRtRows * WORDS;
      for (int i = first; i < kRtRows * GW; i += nthreads) qd[i] = i < nrows * GW ? __ldg(qc_u + (long long)tb * GW + i) : 0u;
      for (int i = first; i < kRtRows * WORDS; i += nthreads) kd[i] = i < nrows * WORDS ? __ldg(kc_u + (long long)tb * WORDS + i) : 0u;
    };
    // Operand A from buffer `buf`: row r = step r of the block, columns -2^13 u_t (sum over the group's heads of
    // -+2^13 per bit, exact in packed bf16 adds), then the three key columns 128, 1, G K 2^13.
    auto build_a = [&](int buf, int nrows, int first, int nthreads) {
      const uint32_t* qd = qraw + buf * kRtRows * GW;
      if (FP8) {  // 16 columns per 16-byte chunk; sums in f16, whose high bytes are the e5m2 values
        constexpr int NC = KB / 16;
        for (int item = first; item < kRtRows * (NC + 1); item += nthreads) {
          const int r = item / (NC + 1), c = item % (NC + 1);
          uint4 v = make_uint4(0u, 0u, 0u, 0u);
          if (c < NC) {
            if (r < nrows) {
              const int w = c >> 1, sh = (c & 1) * 16;
              __half2 sm[8];
#pragma unroll
              for (int k = 0; k < 8; ++k) sm[k] = __float2half2_rn(0.f);
              for (int g = 0; g < G; ++g) {
                const uint32_t bits = qd[r * GW + g * WORDS + w] >> sh;
#pragma unroll
                for (int nb = 0; nb < 4; ++nb) {
                  const uint2 e = s_lut_a[(bits >> (4 * nb)) & 15u];
                  sm[2 * nb] = __hadd2(sm[2 * nb], *reinterpret_cast<const __half2*>(&e.x));
                  sm[2 * nb + 1] = __hadd2(sm[2 * nb + 1], *reinterpret_cast<const __half2*>(&e.y));
                }
              }
              uint32_t wv[4];
#pragma unroll
              for (int k = 0; k < 4; ++k)
                wv[k] = __byte_perm(*reinterpret_cast<uint32_t*>(&sm[2 * k]), *reinterpret_cast<uint32_t*>(&sm[2 * k + 1]), 0x7531);
              v = make_uint4(wv[0], wv[1], wv[2], wv[3]);
            }
            *reinterpret_cast<uint4*>(As + rt_swz(r, c)) = v;
          } else {
            if (r < nrows) v = make_uint4(0x74u | (0x6Cu << 8) | (0x5Cu << 16) | (0x4Cu << 24), 0x3Cu, 0u, 0u);  // 2^14, 4096, 256, 16, 1
            *reinterpret_cast<uint4*>(As + rt_swz(r, XCHUNK)) = v;
            *reinterpret_cast<uint4*>(As + rt_swz(r, XCHUNK + 1)) = make_uint4(0u, 0u, 0u, 0u);
          }
        }
      } else {
      for (int item = first; item < kRtRows * (KB / 8 + 1); item += nthreads) {
        const int r = item / (KB / 8 + 1), c = item % (KB / 8 + 1);
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (c < KB / 8) {
          if (r < nrows) {
            const int w = c >> 2, sh = (c & 3) * 8;
            __nv_bfloat162 s0 = __float2bfloat162_rn(0.f), s1 = s0, s2 = s0, s3 = s0;
            for (int g = 0; g < G; ++g) {
              const uint32_t byte = qd[r * GW + g * WORDS + w] >> sh;
              const uint2 lo = s_lut_a[byte & 15u], hi = s_lut_a[(byte >> 4) & 15u];
              s0 = __hadd2(s0, *reinterpret_cast<const __nv_bfloat162*>(&lo.x));
              s1 = __hadd2(s1, *reinterpret_cast<const __nv_bfloat162*>(&lo.y));
              s2 = __hadd2(s2, *reinterpret_cast<const __nv_bfloat162*>(&hi.x));
              s3 = __hadd2(s3, *reinterpret_cast<const __nv_bfloat162*>(&hi.y));
            }
            v = make_uint4(*reinterpret_cast<uint32_t*>(&s0), *reinterpret_cast<uint32_t*>(&s1),
                           *reinterpret_cast<uint32_t*>(&s2), *reinterpret_cast<uint32_t*>(&s3));
          }
          *reinterpret_cast<uint4*>(As + (c >> 3) * kRtAtomBytes + rt_swz(r, c & 7)) = v;
        } else {
          if (r < nrows) v = make_uint4(0x4300u | (0x3F80u << 16), kconst_bits, 0u, 0u);
          *reinterpret_cast<uint4*>(As + XATOM * kRtAtomBytes + rt_swz(r, XCHUNK)) = v;
          *reinterpret_cast<uint4*>(As + XATOM * kRtAtomBytes + rt_swz(r, XCHUNK + 1)) = make_uint4(0u, 0u, 0u, 0u);
        }
      }
      }
    };
    int t0 = C, cur = 0;
    bool staged = false;  // buffer `cur` and operand A already hold the block that starts at t0
    while (t0 < N) {
      const int rows = (N - t0) < kRtRows ? (N - t0) : kRtRows;
      if (!staged) {  // first block of a unit, or the block before was cut short
        stage_codes(cur, t0, rows, tid, NT);
        __syncthreads();
        build_a(cur, rows, tid, NT);
        fence_proxy_async();
        __syncthreads();
      }
      const uint32_t* qb = qraw + cur * kRtRows * GW;
      const uint32_t* kb_codes = kraw + cur * kRtRows * WORDS;
      // ---- tiles 0 .. nbase-1: base slots; tile nbase: the block's own keys
      const int ntile = nbase + 1;
      const int nsync = (ntile + TP - 1) / TP;
      if (warp >= 4 && warp < kRtMmaWarp) {
        // owner table cleared (-1: the slot still holds its base token); read only by the resolver
        for (int i = tid - 128; i < a.smem_slots / 2; i += 256) reinterpret_cast<uint32_t*>(owner)[i] = 0xFFFFFFFFu;
        // two groups of four warps, one per operand stage: group g expands the tiles that go to stage g
        const int x = (tid - 128) & 127, grp = (tid - 128) >> 7;  // x: this thread's row of the tile
        // Tables in global memory: a group's next base tile (two tiles on) is requested before this tile's wait and
        // expansion, so the L2 latency of the code words is off the group's critical path. The table does not change
        // during a block's tile phase.
        uint32_t hn[WORDS];
        auto fetch_next = [&](int i2) {
          const int j2 = i2 * kRtTile + x;
#pragma unroll
          for (int w = 0; w < WORDS; ++w) hn[w] = (i2 < nbase && j2 < C) ? table_word(j2 * WORDS + w) : 0u;
        };
        if (GLOBAL_TABLE) fetch_next(TP == 1 ? ((it & 1) == grp ? 0 : 1) : grp);
        for (int p = 0; p < nsync; ++p) {
          const int n = it + p, ss = n % NSYNC, ph = (n / NSYNC) & 1;
          if (TP == 1 && (n & 1) != grp) continue;
          const int i = TP == 1 ? p : p * TP + grp;  // this group's tile of the hand-over
          uint32_t hc[WORDS];
          if (GLOBAL_TABLE) {
#pragma unroll
            for (int w = 0; w < WORDS; ++w) hc[w] = hn[w];
            fetch_next(i + 2);
          }
          if (!__all_sync(0xFFFFFFFFu, mbar_wait(empty_bar(ss), ph ^ 1, &abort_flag))) break;
          if (i >= ntile) {  // the block's last hand-over is half empty
            if (lane == 0) mbar_arrive(full_bar(ss));
            continue;
          }
          const int st = TP == 1 ? ss : ss * TP + grp;
          unsigned char* bt = Bs + st * ATOMS * kRtAtomBytes;
          uint32_t h[WORDS];
          bool valid;
          int idx;
          if (i < nbase) {
            const int j = i * kRtTile + x;
            valid = j < C;
            idx = kRtIdxMask - j;
#pragma unroll
            for (int w = 0; w < WORDS; ++w) h[w] = GLOBAL_TABLE ? hc[w] : (valid ? table_word(j * WORDS + w) : 0u);
          } else {  // the block's own keys: plain distances, no index term
            valid = x < rows;
            idx = 0;
#pragma unroll
            for (int w = 0; w < WORDS; ++w) h[w] = kb_codes[x * WORDS + w];
          }
          const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
          unsigned char* brow = bt + (x >> 3) * 1024 + (x & 7) * 128;  // this row inside each swizzle atom
          const int xs = (x & 7) << 4;
          if (FP8) {
            if (valid) {
#pragma unroll
              for (int c = 0; c < KB / 16; ++c) {
                const uint32_t two = h[c >> 1] >> ((c & 1) * 16);
                const uint2 lo = s_lut_b8[two & 0xFFu], hi = s_lut_b8[(two >> 8) & 0xFFu];
                *reinterpret_cast<uint4*>(brow + ((c << 4) ^ xs)) = make_uint4(lo.x, lo.y, hi.x, hi.y);
              }
              *reinterpret_cast<uint4*>(brow + ((XCHUNK << 4) ^ xs)) =
                  make_uint4(cst_e4m3 | (rt_e4m3_of_int(idx >> 12) << 8) | (rt_e4m3_of_int((idx >> 8) & 15) << 16) |
                                 (rt_e4m3_of_int((idx >> 4) & 15) << 24),
                             rt_e4m3_of_int(idx & 15), 0u, 0u);
            } else {
#pragma unroll
              for (int c = 0; c <= KB / 16; ++c) *reinterpret_cast<uint4*>(brow + ((c << 4) ^ xs)) = zero;
            }
          } else if (valid) {
#pragma unroll
            for (int c = 0; c < KB / 8; ++c) {
              const uint32_t byte = h[c >> 2] >> ((c & 3) * 8);
              const uint2 lo = s_lut_b[byte & 15u], hi = s_lut_b[(byte >> 4) & 15u];
              *reinterpret_cast<uint4*>(brow + (c >> 3) * kRtAtomBytes + (((c & 7) << 4) ^ xs)) = make_uint4(lo.x, lo.y, hi.x, hi.y);
            }
            *reinterpret_cast<uint4*>(brow + XATOM * kRtAtomBytes + ((XCHUNK << 4) ^ xs)) =
                make_uint4(rt_bf16_of_int(idx >> 7) | (rt_bf16_of_int(idx & 127) << 16), 0x3F80u, 0u, 0u);
          } else {  // a row past the budget (or past the block's steps): all zeros, its key is 0
#pragma unroll
            for (int c = 0; c < KB / 8; ++c) *reinterpret_cast<uint4*>(brow + (c >> 3) * kRtAtomBytes + (((c & 7) << 4) ^ xs)) = zero;
            *reinterpret_cast<uint4*>(brow + XATOM * kRtAtomBytes + ((XCHUNK << 4) ^ xs)) = zero;
          }
          *reinterpret_cast<uint4*>(brow + XATOM * kRtAtomBytes + (((XCHUNK + 1) << 4) ^ xs)) = zero;
          fence_proxy_async();  // every writing thread orders its stores before the async proxy, then one arrival per warp
          __syncwarp();
          if (lane == 0) mbar_arrive(full_bar(ss));
        }
      } else if (warp == kRtMmaWarp) {
        if (lane == 0) {
          const uint64_t a_desc0 = umma_desc_k128(smem_u32(As));
          for (int p = 0; p < nsync; ++p) {
            const int n = it + p, ss = n % NSYNC, ph = (n / NSYNC) & 1;
            // the readers have drained these accumulators and the expanders have written these operand stages
            if (!mbar_wait2(tempty_bar(ss), ph ^ 1, full_bar(ss), ph, &abort_flag)) break;
            tc_fence_after();
#pragma unroll
            for (int hf = 0; hf < TP; ++hf) {
              if (p * TP + hf >= ntile) break;
              const int st = ss * TP + hf;
              const uint64_t b_desc0 = umma_desc_k128(smem_u32(Bs + st * ATOMS * kRtAtomBytes));
              const uint32_t d_tmem = tmem_base + (uint32_t)(st * kRtTile);
#pragma unroll
              for (int ks = 0; ks < KSTEPS; ++ks) {
                if (FP8) {  // 32 one-byte columns per instruction
                  tc_mma_f8(d_tmem, a_desc0 + (uint64_t)((ks * 32) >> 4), b_desc0 + (uint64_t)((ks * 32) >> 4), idesc, ks > 0);
                } else {
                  const uint32_t off = (uint32_t)(((ks * 16) / 64) * kRtAtomBytes + ((ks * 16) % 64) * 2);
                  tc_mma_bf16(d_tmem, a_desc0 + (uint64_t)(off >> 4), b_desc0 + (uint64_t)(off >> 4), idesc, ks > 0);
                }
              }
            }
            // one commit serves both consumers: when these MMAs are done the accumulators are complete (readers) and the
            // operand stages may be rewritten (expanders); stages and accumulators share the index, so they share the barrier
            tc_commit(tfull_bar(ss));
          }
        }
      } else {
        bool ok = true;
        for (int p = 0; p < nsync && ok; ++p) {
          const int n = it + p, ss = n % NSYNC, ph = (n / NSYNC) & 1;
          ok = __all_sync(0xFFFFFFFFu, mbar_wait(tfull_bar(ss), ph, &abort_flag));
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int hf = 0; hf < TP; ++hf) {
          const int i = p * TP + hf;
          if (i >= ntile) break;
          const bool last_of_handover = hf == TP - 1 || i + 1 >= ntile;  // the accumulators go back after their last read
          const int st = ss * TP + hf;
          const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(st * kRtTile);
          if (i < nbase) {  // the tile's largest key for this step (keys are non-negative floats: compare the bits)
            float mxf, mxs = 0.f;
            if (second) {
              // largest and second-largest key of the tile for this step: four running (first, second) pairs, two
              // elements per update (five instructions), merged at the end. Keys of valid rows are distinct.
              uint32_t v0[32], v1[32], v2[32];
              float f4[4] = {0.f, 0.f, 0.f, 0.f}, s4[4] = {0.f, 0.f, 0.f, 0.f};
              auto upd = [&](int q, float x, float y) {
                const float hi = fmaxf(x, y), lo = fminf(x, y);
                s4[q] = rt_fmax3(s4[q], fminf(f4[q], hi), lo);
                f4[q] = fmaxf(f4[q], hi);
              };
              tc_ld32(taddr, v0);
              tc_ld32(taddr + 32, v1);
              tc_ld32(taddr + 64, v2);
              tc_wait_ld();
#pragma unroll
              for (int k = 0; k < 32; k += 2) upd((k >> 1) & 3, __uint_as_float(v0[k]), __uint_as_float(v0[k + 1]));
              tc_ld32(taddr + 96, v0);
#pragma unroll
              for (int k = 0; k < 32; ++k) upd(k & 3, __uint_as_float(v1[k]), __uint_as_float(v2[k]));
              tc_wait_ld();
#pragma unroll
              for (int k = 0; k < 32; k += 2) upd((k >> 1) & 3, __uint_as_float(v0[k]), __uint_as_float(v0[k + 1]));
              const float fa = fmaxf(f4[0], f4[1]), sa = rt_fmax3(fminf(f4[0], f4[1]), s4[0], s4[1]);
              const float fb = fmaxf(f4[2], f4[3]), sb2 = rt_fmax3(fminf(f4[2], f4[3]), s4[2], s4[3]);
              mxf = fmaxf(fa, fb);
              mxs = rt_fmax3(fminf(fa, fb), sa, sb2);
            } else
            {  // three loads in flight, the fourth issued before the first three are reduced: one exposed load latency per
               // tile. The keys are non-negative whole numbers in fp32, so the floating-point maximum (three inputs per
               // instruction, full-rate pipe) orders them like the integer one (two inputs, half rate); four running
               // maxima keep the reduction from being one chain of dependent instructions.
              uint32_t v0[32], v1[32], v2[32];
              float m4[4] = {0.f, 0.f, 0.f, 0.f};
              tc_ld32(taddr, v0);
              tc_ld32(taddr + 32, v1);
              tc_ld32(taddr + 64, v2);
              tc_wait_ld();
#pragma unroll
              for (int k = 0; k < 32; k += 2) m4[(k >> 1) & 3] = rt_fmax3(m4[(k >> 1) & 3], __uint_as_float(v0[k]), __uint_as_float(v0[k + 1]));
              tc_ld32(taddr + 96, v0);
#pragma unroll
              for (int k = 0; k < 32; ++k) m4[k & 3] = rt_fmax3(m4[k & 3], __uint_as_float(v1[k]), __uint_as_float(v2[k]));
              tc_wait_ld();
#pragma unroll
              for (int k = 0; k < 32; k += 2) m4[(k >> 1) & 3] = rt_fmax3(m4[(k >> 1) & 3], __uint_as_float(v0[k]), __uint_as_float(v0[k + 1]));
              mxf = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
            }
            if (last_of_handover) {
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(tempty_bar(ss));
            }
            Mx[tid * mp + i] = __float2int_rn(mxf);
            if (second) Mx2[tid * mp + i] = __float2int_rn(mxs);
          } else {  // distances of the block's keys: key / 2^14, kept as 16-bit integers
            // ... and, for step `tid`, the largest distance to any key that enters before it (entries e < tid): whatever
            // their slots turn out to be, no new entry's key exceeds (that distance, lowest possible slot)
            float dmax = -1.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              uint32_t v[32];
              tc_ld32(taddr + c * 32, v);
              tc_wait_ld();
              if (kRuns && s_fast) {
#pragma unroll
                for (int k = 0; k < 32; ++k)
                  if (c * 32 + k < tid) dmax = fmaxf(dmax, __uint_as_float(v[k]));
              }
              uint32_t pk[16];
#pragma unroll
              for (int k = 0; k < 16; ++k)
                pk[k] = (uint32_t)__float2int_rn(__uint_as_float(v[2 * k]) * (1.f / 16384.f)) |
                        ((uint32_t)__float2int_rn(__uint_as_float(v[2 * k + 1]) * (1.f / 16384.f)) << 16);
              uint4* dst = reinterpret_cast<uint4*>(Dn + tid * kRtRows + c * 32);
#pragma unroll
              for (int k = 0; k < 4; ++k) dst[k] = make_uint4(pk[4 * k], pk[4 * k + 1], pk[4 * k + 2], pk[4 * k + 3]);
            }
            UB[tid] = dmax < 0.f ? -1 : ((__float2int_rn(dmax * (1.f / 16384.f)) << kRtKeyShift) | kRtIdxMask);
            if (last_of_handover) {
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(tempty_bar(ss));
            }
          }
          }
        }
        if (ok) {
          int rb = 0;
          for (int i = 0; i < nbase; ++i) rb = max(rb, Mx[tid * mp + i]);
          RB[tid] = rb;
        }
        if (kRuns && s_fast) asm volatile("bar.sync 2, 128;" ::: "memory");  // the four reader warps: RB and UB are complete
        if (kRuns && ok && s_fast) {
          // what the resolver's easy-run test needs of step `tid`, in one word: the slot of its best base key (14 bits),
          // whether a new entry might beat that key (bit 14), and how many steps back the nearest earlier step with the
          // same slot lies (bits 16-20; 0: none among the 31 steps before it)
          const int mine = RB[tid] & kRtIdxMask;
          int back = 0;
          for (int q = 1; q < 32 && q <= tid; ++q)
            if (back == 0 && (RB[tid - q] & kRtIdxMask) == mine) back = q;
          PS[tid] = (kRtIdxMask - mine) | (RB[tid] <= UB[tid] ? (1 << 14) : 0) | (back << 16);
        }
      }
      it += nsync;
      tc_fence_before();
      __syncthreads();
      tc_fence_after();
      if (abort_flag) {
        aborted = true;
        break;
      }
      // ---- the block's steps in order (warp 0); meanwhile the other warps prepare the next block's codes and
      // operand A, which do not depend on this block's outcome (only on where the next block starts)
      const int tn = t0 + rows;
      if (warp == 0) {
        // Lane l keeps the block's new entries e = 4l .. 4l+3 as the index half of their keys (16383 - slot), or a
        // large negative number while absent or evicted. Everything a step reads that does not depend on the step
        // before it (its row of new-entry distances, its best base key and that slot's owner, its key code) is
        // fetched one step ahead, so the chain from step to step is a few integer operations and one warp reduction.
        // The two rare cases (a stale base maximum, the scoring pass of the prompt's last step) leave the hot loop,
        // are dealt with outside it and re-enter at the same step: the loop body stays small for the compiler.
        constexpr int kAbsent = -(1 << 30);
        int vb0 = kAbsent, vb1 = kAbsent, vb2 = kAbsent, vb3 = kAbsent;
        int done = rows, stale = 0;
        uint2 dd = *reinterpret_cast<const uint2*>(Dn + 4 * lane);
        int kb = RB[0];
        int own_kb = -1;  // nothing has been evicted yet; >= 0 means: this key's slot may not be taken, repair first
        const int S = cfg.n_sink, Rn = cfg.n_recent;
        // Is the token in `slot` protected at step t? With the ring: `first` = 1 leaves out the token of step t - 1, whose
        // slot is not in the ring yet when the check runs one step ahead (the caller patches that case itself).
        auto protected_at = [&](int slot, int t, int first) -> bool {
          if (GLOBAL_TABLE) {
            const int k = (t - 1 - lane) & 31;
            return slot < S || __any_sync(0xFFFFFFFFu, myring == slot && k >= first && k < Rn);
          }
          const int p = pos_t[slot];
          return p < S || p >= t - Rn;
        };
        if (PROT && protected_at(kRtIdxMask - (kb & kRtIdxMask), t0, 0)) own_kb = 0;
        uint32_t kc[WORDS];
#pragma unroll
        for (int w = 0; w < WORDS; ++w) kc[w] = kb_codes[w];
        bool scored = !(write_scores && t0 + rows == N);  // only the prompt's last step stores Eq. 5 scores
        // Without protected windows most steps need no step-to-step chain at all. A step is EASY when its best base key
        // beats every key a new entry could have (UB) and that base slot still holds its base token: its victim is then
        // that slot, known from the tile maxima alone. Consecutive easy steps with distinct slots do not influence one
        // another (each only removes its own slot and adds an entry the later bounds already cover), so a run of up to 32
        // of them is settled by the warp's lanes side by side. Only the other steps - a stale maximum, a new entry that
        // may win, the scoring pass - go through the sequential path below, one at a time.
        // The run test costs about as much as a sequential step and fails at every step that is not easy, so it only
        // pays while those are few (measured break-even: three steps in ten). A unit starts in the sequential loop, which
        // counts the steps it can tell were not easy; a run-based block counts them exactly, and the unit's next block
        // picks its loop by that count (a run-based block that did not pay holds the unit in the sequential loop for a
        // growing number of blocks). s_fast also tells the readers whether the next block needs the run test's tables
        // (UB, PS) at all.
        const bool FAST = kRuns && s_fast != 0;
        int n_not_easy = 0;
        // the loop is compiled in separate forms, so that the plain sequential one keeps the tight code it had before the run test
        auto resolve_block = [&](auto fast_c, auto count_c) {
          constexpr bool FASTC = decltype(fast_c)::value, COUNT = decltype(count_c)::value;
          bool resume = false;  // re-entering the sequential path at the same step after a repair or the scoring pass
          bool vb_dirty = false;
          if (FASTC) {  // no entry of this block is resident yet
            *reinterpret_cast<int4*>(ES + 4 * lane) = make_int4(kAbsent, kAbsent, kAbsent, kAbsent);
            __syncwarp();
          }
          int r = 0;
          while (r < rows) {
            int status = 0, kn_out = 0;
            if (FASTC && !resume) {
              if (vb_dirty) {  // the sequential path changed the residency of this lane's entries
                *reinterpret_cast<int4*>(ES + 4 * lane) = make_int4(vb0, vb1, vb2, vb3);
                vb_dirty = false;
                __syncwarp();
              }
              for (;;) {
                const int rr = r + lane;
                const bool in = rr < rows;
                const int pk = PS[in ? rr : 0];
                const int sl = pk & kRtIdxMask, back = pk >> 16;
                const int own = owner[sl];
                // not easy: a new entry might win, the slot is no longer its base token's, an earlier step of this run
                // takes the same slot, or this is the prompt's last step and it still has to store its scores
                const bool hard = !in | ((pk >> 14) & 1) | (own >= 0) | (back != 0 && back <= lane) | (!scored && rr == rows - 1) |
                                  !HE_IN_RANGE(sl, C);
                const unsigned hb = __ballot_sync(0xFFFFFFFFu, hard);
                const int ne = hb ? __ffs(hb) - 1 : 32;
                if (ne == 0) break;
                if (lane < ne) {  // Algorithm 1 lines 2-5 on the table for step rr; its token enters as entry rr
                  owner[sl] = (int16_t)rr;
  #pragma unroll
                  for (int w = 0; w < WORDS; ++w) codes_t[sl * WORDS + w] = kb_codes[rr * WORDS + w];
                  pos_t[sl] = t0 + rr;
                  ES[rr] = kRtIdxMask - sl;
                }
                r += ne;
                if (GLOBAL_TABLE) __threadfence_block();
                __syncwarp();
                if (r >= rows) break;
              }
              if (r >= rows) break;
              ++n_not_easy;
              // step r takes the sequential path: its operands, and this lane's entries as the runs left them
              dd = *reinterpret_cast<const uint2*>(Dn + r * kRtRows + 4 * lane);
              kb = RB[r];
              own_kb = owner[kRtIdxMask - (kb & kRtIdxMask)];
  #pragma unroll
              for (int w = 0; w < WORDS; ++w) kc[w] = kb_codes[r * WORDS + w];
              const int4 e4 = *reinterpret_cast<const int4*>(ES + 4 * lane);
              vb0 = e4.x, vb1 = e4.y, vb2 = e4.z, vb3 = e4.w;
            }
            vb_dirty = true;
            resume = false;
            const int r_end = FASTC ? r + 1 : rows;
            // unrolled by two: the carried values (next row's prefetches) change names instead of being copied, which is
            // worth 10-20 % of the loop on this single-warp critical path (measured; unrolling by four is slower again)
  #pragma unroll 2
            for (; r < r_end; ++r) {
              const int rn = r + 1 < rows ? r + 1 : r;  // the last step fetches its own row again (unused)
              const uint2 dd_n = *reinterpret_cast<const uint2*>(Dn + rn * kRtRows + 4 * lane);
              const int kb_n = RB[rn];
              int own_n = owner[kRtIdxMask - (kb_n & kRtIdxMask)];
              int act_slot = 0;
              if (PROT) {  // eligibility of the next step's best base slot at that step; the slot of the entry that turns eligible
                if (protected_at(kRtIdxMask - (kb_n & kRtIdxMask), t0 + r + 1, 1)) own_n = 0;
                if (Rn > 0 && r >= Rn) act_slot = entry_slot[r - Rn];
              }
              uint32_t kc_n[WORDS];
  #pragma unroll
              for (int w = 0; w < WORDS; ++w) kc_n[w] = kb_codes[rn * WORDS + w];
              // best new entry (inserted by an earlier step of this block and still resident)
              const int k0 = (int)((dd.x & 0xFFFFu) << kRtKeyShift) + vb0;
              const int k1 = (int)((dd.x >> 16) << kRtKeyShift) + vb1;
              const int k2 = (int)((dd.y & 0xFFFFu) << kRtKeyShift) + vb2;
              const int k3 = (int)((dd.y >> 16) << kRtKeyShift) + vb3;
              const int kn = __reduce_max_sync(0xFFFFFFFFu, max(max(k0, k1), max(k2, k3)));
              if (COUNT && !FASTC) n_not_easy += (own_kb >= 0 || kn >= kb) ? 1 : 0;  // (a repaired step re-enters and counts twice)
              // best base slot: the tile maxima are upper bounds; one that points at an evicted slot needs a repair
              if (kb > kn && own_kb >= 0) {
                status = 1;
                kn_out = kn;
                break;
              }
              if (!scored && r == rows - 1) {
                status = 2;
                break;
              }
              const int best = max(kb, kn);
              const int slot = kRtIdxMask - (best & kRtIdxMask);
              // a new entry that wins leaves: its lane recognises its own key (keys of resident entries are distinct,
              // absent ones are negative); then this step's token enters as entry r
              // (with protected windows: the entry of step r - n_recent, which is no longer recent from the next step on)
              const int e_act = PROT ? r - Rn : r;
              const bool mine = e_act >= 0 && lane == (e_act >> 2);
              const int sel = e_act & 3, nv = kRtIdxMask - ((PROT && Rn > 0) ? act_slot : slot);
              if (PROT) entry_slot[r] = (uint16_t)slot;
              if (PROT && GLOBAL_TABLE && lane == ((t0 + r) & 31)) myring = slot;
              vb0 = (mine && sel == 0) ? nv : (k0 == best ? kAbsent : vb0);
              vb1 = (mine && sel == 1) ? nv : (k1 == best ? kAbsent : vb1);
              vb2 = (mine && sel == 2) ? nv : (k2 == best ? kAbsent : vb2);
              vb3 = (mine && sel == 3) ? nv : (k3 == best ? kAbsent : vb3);
              // Algorithm 1 lines 2-5 on the table (K / V rows follow in the gather kernel). Every lane stores the same
              // values to the same addresses: no divergent branch, and each lane later reads back its own stores.
              if (HE_IN_RANGE(slot, C)) {
                owner[slot] = (int16_t)r;
  #pragma unroll
                for (int w = 0; w < WORDS; ++w) codes_t[slot * WORDS + w] = kc[w];
                pos_t[slot] = t0 + r;
              }
              if (slot == kRtIdxMask - (kb_n & kRtIdxMask)) own_n = r;  // the owner fetched ahead predates this step
              dd = dd_n, kb = kb_n, own_kb = own_n;
  #pragma unroll
              for (int w = 0; w < WORDS; ++w) kc[w] = kc_n[w];
            }
            if (status != 0) resume = true;
            if (status == 1) {
              // Repair for step r: recompute the maximum of the tile the stale key came from, over the slots that
              // still hold their base token, until the row's best base key is exact (or no longer matters). Each pass
              // makes one tile exact, so nbase passes always suffice; the bound only guards against a corrupted table.
              uint32_t qw[kMaxGroup * WORDS];
  #pragma unroll
              for (int i = 0; i < kMaxGroup * WORDS; ++i) qw[i] = i < GW ? qb[r * GW + i] : 0u;
              const int kn = kn_out;  // the step's best new entry, as the hot loop left it
              // lane i keeps tile i's maximum for this step in a register (tables in shared memory: at most 32 tiles)
              int mt = (!GLOBAL_TABLE && lane < nbase) ? Mx[r * mp + lane] : 0;
              // First the cheap way: the stale key was its tile's largest at the block's start, so the tile's second-largest
              // key bounds what is left of that tile, and it is exact if its slot still holds its base token. If the
              // row's best key is then a live slot (or no better than the best new entry) the step is settled without
              // recomputing a tile.
              bool settled = false;
              if (second) {
                const int cb0 = (kRtIdxMask - (kb & kRtIdxMask)) / kRtTile;
                mt = lane == cb0 ? Mx2[r * mp + cb0] : mt;
                kb = __reduce_max_sync(0xFFFFFFFFu, mt);
                if (kb <= kn) {
                  settled = true;
                } else if (kb > 0) {
                  const int sb = kRtIdxMask - (kb & kRtIdxMask);
                  bool bad = owner[sb] >= 0;
                  if (PROT && !bad) {
                    const int pb = table_pos(sb);
                    bad = pb < S || pb >= t0 + r - Rn;
                  }
                  settled = !bad;
                }
              }
              for (int pass = 0; !settled && pass <= nbase; ++pass) {
                ++stale;
                const int cb = (kRtIdxMask - (kb & kRtIdxMask)) / kRtTile;
                uint32_t hw[kRtTile / 32][WORDS];
                int ow[kRtTile / 32];  // < 0: the slot still holds its base token (and, PROT, that token is eligible now)
  #pragma unroll
                for (int i = 0; i < kRtTile / 32; ++i) {
                  const int j = cb * kRtTile + lane + 32 * i;  // below smem_slots: rows past the budget hold zeros
                  ow[i] = j < C ? (int)owner[j] : 0;
                  if (PROT && j < C) {
                    const int pj = table_pos(j);
                    if (pj < S || pj >= t0 + r - Rn) ow[i] = 0;
                  }
  #pragma unroll
                  for (int w = 0; w < WORDS; ++w) hw[i][w] = j < C ? table_word(j * WORDS + w) : 0u;
                }
                int km = 0;
  #pragma unroll
                for (int i = 0; i < kRtTile / 32; ++i) {
                  int D = 0;
  #pragma unroll
                  for (int g = 0; g < kMaxGroup; ++g) {
                    if (g < G) {
  #pragma unroll
                      for (int w = 0; w < WORDS; ++w) D += __popc(hw[i][w] ^ qw[g * WORDS + w]);
                    }
                  }
                  const int key = (D << kRtKeyShift) + (kRtIdxMask - (cb * kRtTile + lane + 32 * i));
                  km = max(km, ow[i] < 0 ? key : 0);
                }
                km = __reduce_max_sync(0xFFFFFFFFu, km);
                int rowmax;
                if (GLOBAL_TABLE) {
                  Mx[r * mp + cb] = km;  // same value from every lane
                  rowmax = 0;
                  for (int i = lane; i < nbase; i += 32) rowmax = max(rowmax, Mx[r * mp + i]);
                } else {
                  mt = lane == cb ? km : mt;
                  rowmax = mt;
                }
                kb = __reduce_max_sync(0xFFFFFFFFu, rowmax);
                if (kb <= kn) break;
                const int sb = kRtIdxMask - (kb & kRtIdxMask);
                bool bad = owner[sb] >= 0;
                if (PROT && !bad) {
                  const int pb = table_pos(sb);
                  bad = pb < S || pb >= t0 + r - Rn;
                }
                if (!bad) break;
              }
              own_kb = -1;  // exact for this step (or below the best new entry)
              if (stale >= kRtStaleLimit && r + 1 < rows && scored) {  // many repairs: this block ends with step r
                // finish step r here, then stop
                const int best = max(kb, kn);
                const int slot = kRtIdxMask - (best & kRtIdxMask);
                if (HE_IN_RANGE(slot, C)) {
                  owner[slot] = (int16_t)r;
  #pragma unroll
                  for (int w = 0; w < WORDS; ++w) codes_t[slot * WORDS + w] = kc[w];
                  pos_t[slot] = t0 + r;
                }
                if (PROT && GLOBAL_TABLE && lane == ((t0 + r) & 31)) myring = slot;
                done = r + 1;
                break;
              }
            } else if (status == 2) {  // Eq. 5 for every slot as the prompt's last step sees the table
              const uint32_t* qr = qb + r * GW;
              for (int j = lane; j < C; j += 32) {
                uint32_t hj[WORDS];
  #pragma unroll
                for (int w = 0; w < WORDS; ++w) hj[w] = table_word(j * WORDS + w);
                sc[j] = -(float)rt_dist<WORDS>(hj, qr, G);
              }
              scored = true;
            }
          }
        };
        // The kernel with the run-based loop holds one sequential form, which always counts (the count is ignored while
        // the unit is held); a third copy of the loop without the count made the call slower, not faster (code size).
        const bool counting = kRuns && !second && s_hold == 0;
        if (FAST) resolve_block(std::true_type{}, std::true_type{});
        else if (kRuns) resolve_block(std::false_type{}, std::true_type{});
        else resolve_block(std::false_type{}, std::false_type{});
        if (lane == 0) {
          s_done = done;
          // (the sequential loop sees only part of what makes a step not easy, hence its stricter bar for switching back)
          // A run-based block that did not pay sends the unit back to the sequential loop for a number of blocks that
          // doubles with every failure: the sequential loop's own count misses part of what makes a step not easy, so
          // without the hold a unit near the bar would try the run test again every other block.
          bool fast_next;
          if (FAST) {
            fast_next = n_not_easy * kRtFastDen < done * kRtFastNum;
            if (!fast_next) {
              s_backoff = min(4 * s_backoff, 64);
              s_hold = s_backoff;
            } else {
              s_backoff = 2;
            }
          } else if (!counting) {
            if (s_hold > 0) --s_hold;
            fast_next = false;
          } else {
            fast_next = n_not_easy * 10 < done;
          }
          // (with the tiles' second-largest keys at hand the sequential loop settles most stale maxima at once and the run
          // test does not pay: 2.09 against 2.20 ms per call with 1024-slot budgets)
          s_fast = kRuns && !second && fast_next;
        }
      } else if (tn < N) {
        const int nrows = (N - tn) < kRtRows ? (N - tn) : kRtRows;
        stage_codes(cur ^ 1, tn, nrows, tid - 32, NT - 32);
        asm volatile("bar.sync 1, %0;" ::"n"(NT - 32) : "memory");
        build_a(cur ^ 1, nrows, tid - 32, NT - 32);
        fence_proxy_async();
      }
      __syncthreads();
      staged = s_done == rows;  // a block that was cut short restarts from its first unprocessed step
      t0 += s_done;
      if (staged) cur ^= 1;
    }
    if (aborted) break;
    // final state of the unit; everything beyond `fill` is reset
    const bool scored = write_scores && N > C;
    for (int j = tid; j < Cmax; j += NT) {
      const bool valid = j < fill0;
      if (!GLOBAL_TABLE) {
        uint32_t cw[WORDS];
#pragma unroll
        for (int w = 0; w < WORDS; ++w) cw[w] = valid ? codes_t[j * WORDS + w] : 0u;
        store_slot_code<WORDS>(a.cfg, a.ca.codes, unit * Cmax + j, cw);
        a.ca.pos[unit * Cmax + j] = valid ? pos_t[j] : -1;
      }
      if (!(valid && scored)) sc[j] = 0.f;
    }
    if (tid == 0) {
      a.ca.fill[unit] = fill0;
      a.ca.next_pos[unit] = N;
    }
    __syncthreads();  // the tables and s_unit are reused by the next unit
  }

  // A CTA that gave up must not free tensor memory under an MMA that is still writing it (the operands are written by
  // this CTA's own threads, so no copy from outside is ever in flight): one more commit tracks everything the MMA thread
  // has issued, and its completion is awaited (bounded) first.
  if (abort_flag && warp == kRtMmaWarp && lane == 0) {
    const uint32_t drain_bar = bar0 + 8u * (4 * NSTAGE);
    tc_commit(drain_bar);
    mbar_drain(drain_bar, 0);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kRtMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(NSTAGE * kRtTile) : "memory");
  }
  if (tid == 0 && abort_flag) atomicAdd(&g_tc_error, 1);
}

}  // namespace he
