// he_decode_step with HE_FLAG_EARLY_INPUTS, one CTA per SM: Algorithm 1 lines 1-5 for up to four (sequence, KV head)
// units per CTA.
//
// A decode call moves little (15 MB in the "throughput batch" shape) and is a chain of dependent phases: fetch the
// step's rows, project them (Eq. 2), fetch each unit's code table, score it (Eq. 5), reduce (Eq. 6), overwrite the
// slot. Consecutive calls of a stream overlap through programmatic dependent launch, and only the table, the
// positions and the counters can have been written by the call before this one: with the flag the caller promises
// that q, k, v were complete before the call was enqueued, so everything up to the query contexts of Eq. 5 runs BEFORE
// griddepcontrol.wait, under the previous call's scan. What bounds a call is then the part after the wait.
//   * Placement. The grid has one CTA of 512 threads per SM (at most 64 registers and 113 KB of shared memory, so
//     that exactly two calls' CTAs fit an SM). A CTA owns up to four units, dealt out by budget (largest first, in
//     a snake over the CTAs) so that every SM scans about the same number of slots. With one small CTA per unit the
//     hardware placed the CTAs of the next call wherever slots became free first, up to seven on one SM, and the
//     slowest SM set the pace.
//   * Parallelism per unit. All 512 threads scan each of the CTA's units in turn; a thread sees at most four
//     16-byte code vectors of a 4096-slot table. The vectors of all the CTA's units stream through one ring of eight
//     16-byte slots per thread (cp.async, no registers held), each slot copied, read and refilled by its own thread
//     only, so the ring needs no barrier. The tables were asked into L2 before the wait (a prefetch returns no data,
//     so it cannot observe a stale value), which moves the HBM transfer under the previous call's scan.
//   * Nothing after the wait touches the kernel parameters (see SmUnit).
//
// Projection: on tensor cores for bf16 rows (three exact bf16 terms of W, fp32 accumulation), else in the order of
// decode_step_kernel (32-channel fmaf chains in ascending channel order, chunk sums added in ascending chunk order).
#pragma once
#include <type_traits>

#include "common.cuh"
#include "decode_kernels.cuh"

namespace he {

constexpr int kSmThreads = 512;
constexpr int kSmWarps = kSmThreads / 32;
constexpr int kSmUnits = 4;         // units per CTA at most
constexpr int kSmStages = 8;        // 16-byte code vectors in flight per thread
constexpr int kSmRowBatch = 5;      // CUDA-core projection: rows per thread and pass (G = 4 queries + the key)
constexpr int kSmPassRows = 20;     // CUDA-core projection: rows staged per pass (four units of five rows)
constexpr int kSmMmaRows = 40;      // tensor-core projection: staged rows (4 units x 9 rows at most, in tiles of 8)
constexpr int kSmMmaStride = 288;   // ... bytes between staged rows: 256 of data + 32, so that 8-byte fragment reads of a
                                    // half-warp (4 rows x 4 lanes) fall into 32 different banks
constexpr int kSmPartStride = 68;   // ... words between rows of the partial-sum table (conflict-free fragment stores)
constexpr int kSmSchedShift = 21;   // DecodeArgs::sched word = sequence << 21 | budget

struct SmLayout {
  size_t ring, xs, part, kv, total;
};
// Dynamic shared memory. The ring reuses the projection's staging: the projection is over before the wait, the ring
// fills after it.
__host__ __device__ inline SmLayout sm_layout(int d, int words, int es, bool mma) {
  SmLayout L;
  const int nch = (d + kChunk - 1) / kChunk;
  const size_t ring_bytes = (size_t)kSmStages * kSmThreads * 16;
  const size_t xs_bytes = mma ? (size_t)kSmMmaRows * kSmMmaStride : (size_t)kSmPassRows * d * sizeof(float);
  const size_t part_bytes = mma ? (size_t)4 * kSmMmaRows * kSmPartStride * sizeof(float)
                                : (size_t)kSmPassRows * nch * 32 * words * sizeof(float);
  L.ring = 0;
  L.xs = 0;
  L.part = xs_bytes;
  const size_t work = ring_bytes > xs_bytes + part_bytes ? ring_bytes : xs_bytes + part_bytes;
  L.kv = work;
  L.total = work + (size_t)kSmUnits * 2 * d * es;
  return L;
}

// Everything the kernel needs after the wait is resolved before it and kept in shared memory. Kernel parameters live
// in constant memory, every launch has its own copy, and a first touch of one of its lines costs a trip to L2: on the
// critical path after the wait those trips (fill, next_pos, the output pointers, ...) add up.
struct SmUnit {
  const uint4* cvec;   // the unit's code table
  float* sc;           // its scores
  int32_t* pp;         // its positions
  int32_t* fill_p;     // its counters
  int32_t* npos_p;
  int32_t* victim_p;   // its outputs
  int32_t* evpos_p;    // nullable
  char* k_rows;        // its K and V slots
  char* v_rows;
  uint32_t* codes_p;   // its code table, for the slot rewrite
  uint32_t* qcodes_p;  // nullable: where its query codes go
  int unit, C, nvec;
};

// One warp waits for the stream's previous kernel, the others sleep at the barrier. With every warp in
// griddepcontrol.wait the waiting CTA slowed the CTA it shares the SM with.
__device__ __forceinline__ void cta_griddep_wait(int warp) {
  if (warp == 0) griddep_wait();
  __syncthreads();
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                               uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Two fp32 values -> their bf16 roundings packed (x in the low half), and the exact remainders.
__device__ __forceinline__ uint32_t split_bf16x2(float& x, float& y) {
  uint32_t packed;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(packed) : "f"(y), "f"(x));
  x -= __uint_as_float(packed << 16);
  y -= __uint_as_float(packed & 0xFFFF0000u);
  return packed;
}

// MMA = true (bf16 rows, head_dim a multiple of 32 up to 128): Eq. 2 on warp-level tensor-core instructions. The fp32
// W is split on the fly into three bf16 terms whose sum is W exactly, so every product is exact and only the fp32
// accumulation rounds (smallest term first). On CUDA cores the projection of a call's rows was bound by the shared-memory
// reads of the rows (one 16-byte broadcast read per four multiply-adds): 3 us per call of this shape against 0.3 us.
template <int WORDS, int GT, bool MMA>
__global__ void __launch_bounds__(kSmThreads, 2) decode_step_sm_kernel(const DecodeArgs a) {
  constexpr int NT = kSmThreads, NW = kSmWarps;
  constexpr int SPV = 4 / WORDS;  // slots per 16-byte vector
  constexpr int BP = 32 * WORDS;
  using Ctx = QueryCtx<WORDS, GT>;
  extern __shared__ __align__(16) unsigned char ssm[];
  __shared__ SmUnit su[kSmUnits];
  __shared__ he_config cfg_s;
  __shared__ const void* in_s[4];  // q, k, v, W
  __shared__ __align__(16) uint32_t codes_s[kSmUnits][(kMaxGroup + 1) * WORDS];  // per unit: G query codes, then the key code
  __shared__ __align__(16) uint32_t rec_s[kSmUnits][Ctx::kRecWords];
  __shared__ uint32_t wbest[2][kSmUnits][NW];

  // The next call of the stream may start at once: before its own wait it reads nothing that this kernel writes.
  griddep_launch_dependents();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 32) {
    cfg_s = a.cfg;
    in_s[0] = a.q, in_s[1] = a.k, in_s[2] = a.v, in_s[3] = a.ca.W;
  }
  // ---- this CTA's units: rank r of the budget order goes to CTA r % grid in even rounds, mirrored in odd rounds
  if (tid < kSmUnits) {
    const he_config& cfg = a.cfg;
    const int d = cfg.head_dim, G = cfg.group_size, es = esize_of(cfg.dtype), Cmax = cfg.max_budget, H = cfg.n_kv_heads;
    const int units = cfg.batch * H, grid = gridDim.x;
    const int rounds = (units + grid - 1) / grid;
    SmUnit u;
    u.unit = -1;
    u.C = u.nvec = 0;
    if (tid < rounds) {
      const int rank = tid * grid + ((tid & 1) ? grid - 1 - (int)blockIdx.x : (int)blockIdx.x);
      if (rank < units) {
        const int so = rank / H, h = rank - so * H;
        int s = so, C;
        if (a.n_sched > 0) {  // sequences by budget, largest first, with their budgets (from the caller's host mirror)
          const uint32_t sw = a.sched[so];
          s = (int)(sw >> kSmSchedShift);
          C = (int)(sw & ((1u << kSmSchedShift) - 1u));
        } else {
          C = __ldg(a.ca.budget + s);  // read-only while the cache is in use, so it may be read before the wait
        }
        u.unit = s * H + h;
        u.C = max(min(C, Cmax), 0);
        u.nvec = (u.C * WORDS + 3) / 4;
        u.cvec = reinterpret_cast<const uint4*>(a.ca.codes + (size_t)u.unit * Cmax * WORDS);
        u.sc = a.ca.scores + (size_t)u.unit * Cmax;
        u.pp = a.ca.pos + (size_t)u.unit * Cmax;
        u.fill_p = a.ca.fill + u.unit;
        u.npos_p = a.ca.next_pos + u.unit;
        u.victim_p = a.victim_out + u.unit;
        u.evpos_p = a.evicted_pos_out != nullptr ? a.evicted_pos_out + u.unit : nullptr;
        u.k_rows = static_cast<char*>(a.ca.k_cache) + (size_t)u.unit * Cmax * d * es;
        u.v_rows = static_cast<char*>(a.ca.v_cache) + (size_t)u.unit * Cmax * d * es;
        u.codes_p = a.ca.codes + (size_t)u.unit * Cmax * WORDS;
        u.qcodes_p = a.qcodes_out != nullptr ? a.qcodes_out + (size_t)u.unit * G * WORDS : nullptr;
        // the table (and, with protected windows, the positions) is asked into L2 now
        if (u.nvec > 0) {
          l2_prefetch_bulk(u.cvec, (uint32_t)u.nvec * 16u);
          if (cfg.n_sink > 0 || cfg.n_recent > 0) l2_prefetch_bulk(u.pp, (uint32_t)((u.C + 3) / 4) * 16u);
        }
      }
    }
    su[tid] = u;
  }
  if (tid < kSmUnits * (kMaxGroup + 1) * WORDS) (&codes_s[0][0])[tid] = 0u;  // the tensor-core path stores code bytes
  __syncthreads();
  const he_config& cfg = cfg_s;
  const int d = cfg.head_dim, b = cfg.hash_bits, G = cfg.group_size, es = esize_of(cfg.dtype);
  const int Cmax = cfg.max_budget;
  const int R = G + 1;
  const int cpr = d * es / 16;  // 16-byte chunks per row
  const void* const q_in = in_s[0];
  const void* const k_in = in_s[1];
  const void* const v_in = in_s[2];
  const float* const W_in = static_cast<const float*>(in_s[3]);
  const SmLayout L = sm_layout(d, WORDS, es, MMA);
  uint4* ring = reinterpret_cast<uint4*>(ssm + L.ring);
  unsigned char* xs_raw = ssm + L.xs;                    // tensor-core projection: [kSmMmaRows] rows of kSmMmaStride bytes
  float* xs = reinterpret_cast<float*>(ssm + L.xs);      // CUDA-core projection: [kSmPassRows][d]
  float* part = reinterpret_cast<float*>(ssm + L.part);  // ... [kSmPassRows][nch][BP]
  uint4* kvs = reinterpret_cast<uint4*>(ssm + L.kv);     // [kSmUnits][2][cpr]
  const int n_sink = cfg.n_sink, n_recent = cfg.n_recent;
  const uint32_t flags = cfg.flags;
  int n_mine = 0;
#pragma unroll
  for (int i = 0; i < kSmUnits; ++i) n_mine += su[i].unit >= 0 ? 1 : 0;  // valid units come first: a hole can only be in the last round
  const int rows_total = n_mine * R;

  // ---- W (it never changes while a cache is in use)
  const int nch = d / kChunk;  // the host sends only whole chunks here
  // CUDA cores: work item = (chunk of 32 channels, bit); thread groups share the rows between them
  const int nitems = nch * BP;
  const int groups = NT / nitems;
  const int item = tid % nitems, grp = tid / nitems;
  // tensor cores: D[bit][row] = sum_ch W[ch][bit] x[row][ch] with the BITS as the instruction's M (tiles of 16) and the
  // step's rows as its N (tiles of 8): 20 rows are three N-tiles instead of two half-empty M-tiles, and a warp's
  // fragments of W serve all of them. Warp (mt, kq) = (warp % 4, warp / 4) owns bits 16 mt .. 16 mt + 15 and the
  // 16-channel steps kq and kq + 4; lane (g, tg) holds W[16 ks + 4 tg + j][16 mt + g (+ 8)], j < 4: inside a step a
  // lane's four channels stand in for the instruction's k = 2 tg, 2 tg + 1, 2 tg + 8, 2 tg + 9 (the order of the terms
  // of a dot product is free, and the rows are read with the same assignment).
  const int m_tiles = (b + 15) >> 4, mt = warp & 3, kq = warp >> 2, g = lane >> 2, tg = lane & 3;
  const int nks = d >> 4;
  float wreg[MMA ? 16 : kChunk];
  {
    if (MMA) {
#pragma unroll
      for (int h2 = 0; h2 < 2; ++h2) {  // this warp's first and second step
        const int ks = kq + 4 * h2;
#pragma unroll
        for (int hb = 0; hb < 2; ++hb) {  // bit g, bit g + 8
          const int bit = 16 * mt + g + 8 * hb;
          const bool on = mt < m_tiles && ks < nks && bit < b;  // columns beyond b count as zeros
          const float* wb = W_in + (size_t)(16 * ks + 4 * tg) * b + bit;
#pragma unroll
          for (int j = 0; j < 4; ++j) wreg[(h2 * 2 + hb) * 4 + j] = on ? __ldg(wb + j * b) : 0.f;
        }
      }
    } else if (grp < groups) {
      const int c0 = (item / BP) * kChunk, bi = item % BP;
      const float* wp = W_in + (size_t)c0 * b + bi;
      const bool on = bi < b;
#pragma unroll
      for (int cc = 0; cc < kChunk; ++cc) wreg[cc] = on ? __ldg(wp + cc * b) : 0.f;
    }
  }

  // A warp copies a row, a lane 16 bytes of it (no per-thread index arithmetic).
  if (warp < 2 * n_mine) {
    const int i = warp >> 1;
    const bool is_k = (warp & 1) == 0;
    const char* src = static_cast<const char*>(is_k ? k_in : v_in) + (size_t)su[i].unit * d * es;
    for (int ch = lane; ch < cpr; ch += 32) cp_async16(kvs + (i * 2 + (is_k ? 0 : 1)) * cpr + ch, reinterpret_cast<const uint4*>(src) + ch);
  }
  if (MMA) {  // the rows to hash, as they are (bf16)
    for (int p = warp; p < rows_total; p += NW) {
      const int i = p / R, row = p - i * R, unit = su[i].unit;
      const char* src = row < G ? static_cast<const char*>(q_in) + ((size_t)unit * G + row) * d * es
                                : static_cast<const char*>(k_in) + (size_t)unit * d * es;
      for (int ch = lane; ch < cpr; ch += 32) cp_async16(xs_raw + p * kSmMmaStride + ch * 16, reinterpret_cast<const uint4*>(src) + ch);
    }
    // rows that only pad the last tile of 8: zeros (their sums are never read)
    for (int p = rows_total + warp; p < ((rows_total + 7) & ~7); p += NW)
      for (int ch = lane; ch < cpr; ch += 32) *reinterpret_cast<uint4*>(xs_raw + p * kSmMmaStride + ch * 16) = make_uint4(0u, 0u, 0u, 0u);
  }
  cp_async_commit();

  // The code tables stream through a ring of kSmStages 16-byte slots per thread; a thread copies, reads and refills
  // only its own slots.
  // Issue cursor: the unit being copied, this thread's next vector in it and how many it still has there. A thread's
  // slots are 16 bytes each, NT * 16 bytes apart; `rpos` walks them round and round (consume, refill, step).
  int iu = -1, irem = 0;
  const uint4* iptr = nullptr;
  const uint32_t rbase = (uint32_t)__cvta_generic_to_shared(ring + tid);
  constexpr uint32_t kRingMask = kSmStages * NT * 16 - 1;
  auto issue_at = [&](uint32_t saddr) {
    while (irem == 0 && iu + 1 < n_mine) {
      ++iu;
      const int nv = su[iu].nvec;
      irem = nv > tid ? (nv - tid + NT - 1) / NT : 0;
      iptr = su[iu].cvec + tid;
    }
    if (irem > 0) {
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(saddr), "l"(iptr) : "memory");
      iptr += NT;
      --irem;
    }
    cp_async_commit();
  };
  // The first round of the ring is addressed before the wait, so that only the copies themselves follow it.
  const uint4* first[kSmStages];
  auto plan_ring = [&]() {
#pragma unroll
    for (int sl = 0; sl < kSmStages; ++sl) {
      while (irem == 0 && iu + 1 < n_mine) {
        ++iu;
        const int nv = su[iu].nvec;
        irem = nv > tid ? (nv - tid + NT - 1) / NT : 0;
        iptr = su[iu].cvec + tid;
      }
      first[sl] = irem > 0 ? iptr : nullptr;
      if (irem > 0) iptr += NT, --irem;
    }
  };
  auto fill_ring = [&]() {
#pragma unroll
    for (int sl = 0; sl < kSmStages; ++sl) {
      if (first[sl] != nullptr)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(rbase + sl * NT * 16), "l"(first[sl]) : "memory");
      cp_async_commit();
    }
  };
  cp_async_wait_all();  // the staged rows have landed

  // ---- Eq. 2 on the units' G query rows and key row
  if (MMA) {
    __syncthreads();
    const int n_tiles = (rows_total + 7) >> 3;  // at most 5
    if (mt < m_tiles && kq < nks) {
      float acc[5][4];
#pragma unroll
      for (int n = 0; n < 5; ++n)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[n][j] = 0.f;
#pragma unroll
      for (int h2 = 0; h2 < 2; ++h2) {
        const int ks = kq + 4 * h2;
        if (ks >= nks) break;
        // three exact bf16 terms of this step's fragment of W: a0 = (bit g; k 2tg, 2tg+1), a1 = (bit g + 8; same k),
        // a2 = (bit g; k 2tg + 8, + 9), a3 = (bit g + 8; same)
        float w00 = wreg[h2 * 8 + 0], w01 = wreg[h2 * 8 + 1], w02 = wreg[h2 * 8 + 2], w03 = wreg[h2 * 8 + 3];
        float w10 = wreg[h2 * 8 + 4], w11 = wreg[h2 * 8 + 5], w12 = wreg[h2 * 8 + 6], w13 = wreg[h2 * 8 + 7];
        uint32_t at[3][4];
#pragma unroll
        for (int term = 0; term < 3; ++term) {
          at[term][0] = split_bf16x2(w00, w01);
          at[term][1] = split_bf16x2(w10, w11);
          at[term][2] = split_bf16x2(w02, w03);
          at[term][3] = split_bf16x2(w12, w13);
        }
#pragma unroll
        for (int n = 0; n < 5; ++n) {
          if (n >= n_tiles) break;
          // row 8 n + g, channels 16 ks + 4 tg + 0..3: 8 bytes
          const uint2 xv = *reinterpret_cast<const uint2*>(xs_raw + (8 * n + g) * kSmMmaStride + (16 * ks + 4 * tg) * 2);
#pragma unroll
          for (int term = 2; term >= 0; --term)  // smallest term first
            mma_bf16_16816(acc[n], at[term][0], at[term][1], at[term][2], at[term][3], xv.x, xv.y);
        }
      }
      // partial sums of this warp's channel steps: P[kq][row][bit]
#pragma unroll
      for (int n = 0; n < 5; ++n) {
        if (n >= n_tiles) break;
#pragma unroll
        for (int j = 0; j < 4; ++j)
          part[((kq * kSmMmaRows) + 8 * n + 2 * tg + (j & 1)) * kSmPartStride + 16 * mt + g + 8 * (j >> 1)] = acc[n][j];
      }
    }
    __syncthreads();
    // sign bits: a warp takes a row, a lane the bits lane and lane + 32; the steps' partial sums are added in order
    const int nkq = nks < 4 ? nks : 4;
    for (int p = warp; p < rows_total; p += NW) {
      const int i = p / R, row = p - i * R;
#pragma unroll
      for (int w = 0; w < WORDS; ++w) {
        const int bit = 32 * w + lane;
        float tot = 0.f;
        if (bit < 16 * m_tiles)
          for (int q4 = 0; q4 < nkq; ++q4) tot += part[(q4 * kSmMmaRows + p) * kSmPartStride + bit];
        const uint32_t word = __ballot_sync(0xFFFFFFFFu, tot >= 0.f) & word_mask(b, w);
        if (lane == 0) codes_s[i][row * WORDS + w] = word;
      }
    }
    __syncthreads();
  } else {
    for (int p0 = 0; p0 < rows_total; p0 += kSmPassRows) {
      const int prow = min(kSmPassRows, rows_total - p0);
      if (p0 > 0) __syncthreads();
      for (int idx = tid; idx < prow * cpr; idx += NT) {  // rows of the pass as fp32
        const int rr = idx / cpr, ch = idx - rr * cpr;
        const int p = p0 + rr, i = p / R, row = p - i * R;
        const int unit = su[i].unit;
        const char* src = row < G ? static_cast<const char*>(q_in) + ((size_t)unit * G + row) * d * es
                                  : static_cast<const char*>(k_in) + (size_t)unit * d * es;
        store_chunk(xs + rr * d, __ldg(reinterpret_cast<const uint4*>(src) + ch), ch, cfg.dtype);
      }
      __syncthreads();
      if (grp < groups) {
        const int per = (prow + groups - 1) / groups;  // this group's rows of the pass: [r_lo, r_hi)
        const int r_lo = grp * per, r_hi = min(prow, r_lo + per);
        const int qd = item / BP, bi = item % BP;
        const float* xb = xs + qd * kChunk;
        for (int rb = r_lo; rb < r_hi; rb += kSmRowBatch) {
          float acc[kSmRowBatch];
#pragma unroll
          for (int r = 0; r < kSmRowBatch; ++r) acc[r] = 0.f;
#pragma unroll
          for (int cc = 0; cc < kChunk; cc += 4) {
#pragma unroll
            for (int r = 0; r < kSmRowBatch; ++r) {
              // rows beyond the range are read (they lie inside the staging area) and their sums dropped
              const float4 xv = *reinterpret_cast<const float4*>(xb + min(rb + r, kSmPassRows - 1) * d + cc);
              acc[r] = fmaf(xv.x, wreg[cc], acc[r]);
              acc[r] = fmaf(xv.y, wreg[cc + 1], acc[r]);
              acc[r] = fmaf(xv.z, wreg[cc + 2], acc[r]);
              acc[r] = fmaf(xv.w, wreg[cc + 3], acc[r]);
            }
          }
#pragma unroll
          for (int r = 0; r < kSmRowBatch; ++r)
            if (rb + r < r_hi) part[((rb + r) * nch + qd) * BP + bi] = acc[r];
        }
      }
      __syncthreads();
      for (int task = warp; task < prow * WORDS; task += NW) {  // chunk sums -> sign bits, one ballot per word
        const int rr = task / WORDS, w = task - rr * WORDS;
        float tot = 0.f;
        for (int q2 = 0; q2 < nch; ++q2) tot += part[(rr * nch + q2) * BP + 32 * w + lane];
        const uint32_t word = __ballot_sync(0xFFFFFFFFu, tot >= 0.f) & word_mask(b, w);
        const int p = p0 + rr, i = p / R, row = p - i * R;
        if (lane == 0) codes_s[i][row * WORDS + w] = word;
      }
    }
    __syncthreads();
  }
  // the query contexts of Eq. 5, one per unit
  if (warp < n_mine && lane == 0) Ctx::build(rec_s[warp], codes_s[warp], G);
  __syncthreads();

  // ---- everything below may depend on the previous kernel of the stream
  plan_ring();
  cta_griddep_wait(warp);
  fill_ring();
  // counters: every thread reads the fill of its CTA's units itself (no barrier between the wait and the scan); the
  // warp that will finish unit `warp` also keeps that unit's position
  const bool prot = n_sink > 0 || n_recent > 0;
  int fl[kSmUnits], tt[kSmUnits];
#pragma unroll
  for (int i = 0; i < kSmUnits; ++i) {
    fl[i] = i < n_mine ? __ldcg(su[i].fill_p) : 0;
    tt[i] = (i < n_mine && (prot || i == warp)) ? __ldcg(su[i].npos_p) : 0;
  }
  if (su[0].qcodes_p != nullptr)  // (all units or none)
    for (int idx = tid; idx < n_mine * G * WORDS; idx += NT) {
      const int i = idx / (G * WORDS), w = idx - i * G * WORDS;
      su[i].qcodes_p[w] = codes_s[i][w];
    }

  // ---- Eq. 5 / Eq. 6: every thread walks its vectors of each unit in turn; the ring delivers them in that order
  const bool write_scores = (flags & HE_FLAG_WRITE_SCORES) != 0;
  constexpr uint32_t kKeyBase = (1u << kKeyIdxBits) + kKeyIdxMask;  // key = (rank << 20) + kKeyBase - slot
  uint32_t rpos = 0;  // ring position of the next vector to consume
  auto scan = [&](auto prot_c, auto scores_c) {
    constexpr bool PROT = decltype(prot_c)::value, SCORES = decltype(scores_c)::value;
#pragma unroll
    for (int i = 0; i < kSmUnits; ++i) {
      if (i >= n_mine) break;
      const int C = su[i].C, nvec = su[i].nvec, t = tt[i];
      const bool evict = C >= 1 && fl[i] >= C;
      const int nfull = C / SPV;  // vectors whose slots all lie below C; at most one more holds the tail
      const int cfull = nfull > tid ? (nfull - tid + NT - 1) / NT : 0;
      const bool tail = nvec > nfull && ((nvec - 1) & (NT - 1)) == tid;
      uint32_t best_all = 0u, best_el = 0u;
      auto take = [&]() {  // the oldest copy in flight has landed: read it and refill its slot
        cp_async_wait_pending(kSmStages - 1);
        uint4 v;
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(rbase + rpos) : "memory");
        issue_at(rbase + rpos);
        rpos = (rpos + NT * 16) & kRingMask;
        return v;
      };
      if (!evict) {  // a unit that is still filling scores nothing; its copies are consumed all the same
        for (int k = 0; k < cfull + (tail ? 1 : 0); ++k) take();
      } else {
        Ctx ctx;
        ctx.load(rec_s[i], G);
        const int j0 = tid * SPV;
        float* sp = su[i].sc + j0;
        const int32_t* pq = su[i].pp + j0;
        uint32_t kb = kKeyBase - (uint32_t)j0;
        auto score_full = [&](const uint4& cvv) {  // a vector whose slots all count
          const uint32_t wds[4] = {cvv.x, cvv.y, cvv.z, cvv.w};
          int rk[SPV];
#pragma unroll
          for (int e = 0; e < SPV; ++e) {
            uint32_t h[WORDS];
#pragma unroll
            for (int w = 0; w < WORDS; ++w) h[w] = wds[e * WORDS + w];
            rk[e] = ctx.rank(h);
          }
          int pv[4] = {0, 0, 0, 0};
          if (PROT) {
            if (SPV == 4) {
              const int4 q4 = __ldcg(reinterpret_cast<const int4*>(pq));
              pv[0] = q4.x, pv[1] = q4.y, pv[2] = q4.z, pv[3] = q4.w;
            } else {
              const int2 q2 = __ldcg(reinterpret_cast<const int2*>(pq));
              pv[0] = q2.x, pv[1] = q2.y;
            }
          }
#pragma unroll
          for (int e = 0; e < SPV; ++e) {
            const uint32_t key = ((uint32_t)rk[e] << kKeyIdxBits) + (kb - (uint32_t)e);
            best_all = max(best_all, key);
            if (PROT && pv[e] >= n_sink && pv[e] < t - n_recent) best_el = max(best_el, key);
          }
          if (SCORES) {
            if (SPV == 4)
              __stcg(reinterpret_cast<float4*>(sp),
                     make_float4(neg_small_int(ctx.dist(rk[0])), neg_small_int(ctx.dist(rk[1])),
                                 neg_small_int(ctx.dist(rk[SPV > 2 ? 2 : 0])), neg_small_int(ctx.dist(rk[SPV > 3 ? 3 : 0]))));
            else
              __stcg(reinterpret_cast<float2*>(sp), make_float2(neg_small_int(ctx.dist(rk[0])), neg_small_int(ctx.dist(rk[1]))));
          }
          sp += NT * SPV;
          pq += NT * SPV;
          kb -= NT * SPV;
        };
        int k = 0;
        for (; k < cfull; ++k) score_full(take());
        if (tail) {  // the unit's last vector, cut short by the budget: one thread
          const uint4 cvv = take();
          const uint32_t wds[4] = {cvv.x, cvv.y, cvv.z, cvv.w};
          const int jt = nfull * SPV;
#pragma unroll
          for (int e = 0; e < SPV; ++e)
            if (jt + e < C) {
              uint32_t h[WORDS];
#pragma unroll
              for (int w = 0; w < WORDS; ++w) h[w] = wds[e * WORDS + w];
              const int r1 = ctx.rank(h);
              const uint32_t key = ((uint32_t)r1 << kKeyIdxBits) + (kKeyBase - (uint32_t)(jt + e));
              best_all = max(best_all, key);
              if (PROT) {
                const int p = __ldcg(su[i].pp + jt + e);
                if (p >= n_sink && p < t - n_recent) best_el = max(best_el, key);
              }
              if (SCORES) su[i].sc[jt + e] = neg_small_int(ctx.dist(r1));
            }
        }
      }
      best_all = __reduce_max_sync(0xFFFFFFFFu, best_all);
      if (PROT) best_el = __reduce_max_sync(0xFFFFFFFFu, best_el);
      if (lane == 0) {
        wbest[0][i][warp] = best_all;
        if (PROT) wbest[1][i][warp] = best_el;
      }
    }
  };
  using T = std::true_type;
  using F = std::false_type;
  if (prot) {
    if (write_scores) scan(T{}, T{}); else scan(T{}, F{});
  } else {
    if (write_scores) scan(F{}, T{}); else scan(F{}, F{});
  }
  cp_async_wait_all();
  __syncthreads();

  // ---- Algorithm 1 lines 2-5: warp i finishes unit i; the slot takes the new token's K, V, code and position
  if (warp < n_mine) {
    const int i = warp;
    int fill = 0, t = 0;
#pragma unroll
    for (int j = 0; j < kSmUnits; ++j)
      if (j == i) fill = fl[j], t = tt[j];
    const SmUnit& u = su[i];
    const int C = u.C;
    if (C < 1 || !HE_IN_RANGE(fill, Cmax + 1)) {  // a unit without a budget holds nothing: report it and leave the state alone
      if (lane == 0) {
        *u.victim_p = -1;
        if (u.evpos_p != nullptr) *u.evpos_p = -1;
      }
      return;
    }
    const bool evict = fill >= C;
    int slot = min(fill, Cmax - 1);
    if (evict) {
      uint32_t fin = __reduce_max_sync(0xFFFFFFFFu, lane < NW ? wbest[0][i][lane] : 0u);
      if (prot) {
        const uint32_t fin_el = __reduce_max_sync(0xFFFFFFFFu, lane < NW ? wbest[1][i][lane] : 0u);
        if (fin_el != 0u) fin = fin_el;
      }
      slot = min((int)(kKeyIdxMask - (fin & kKeyIdxMask)), C - 1);  // (the clamp never acts on a scored table)
    }
    if (!HE_IN_RANGE(slot, C)) return;
    const size_t row_bytes = (size_t)cpr * 16;
    for (int c = lane; c < 2 * cpr; c += 32) {
      const bool is_k = c < cpr;
      char* dst = (is_k ? u.k_rows : u.v_rows) + (size_t)slot * row_bytes;
      reinterpret_cast<uint4*>(dst)[is_k ? c : c - cpr] = kvs[i * 2 * cpr + c];
    }
    if (lane == 0) {
      int ev = -1;
      if (evict && u.evpos_p != nullptr) ev = __ldcg(u.pp + slot);
      u.pp[slot] = t;
#pragma unroll
      for (int w = 0; w < WORDS; ++w) u.codes_p[(size_t)slot * WORDS + w] = codes_s[i][G * WORDS + w];
      if (!evict) {
        u.sc[slot] = 0.f;
        *u.fill_p = fill + 1;
      }
      *u.npos_p = t + 1;
      *u.victim_p = slot;
      if (u.evpos_p != nullptr) *u.evpos_p = ev;
    }
  }
}

}  // namespace he
