// he_decode_step: Algorithm 1 lines 1-5 for one (sequence, KV head) unit per CTA.
//
// Data flow of one CTA
//   1. the unit's packed code words are copied global -> shared with 16-byte cp.async (no registers held, the
//      copies fly while the new rows are hashed); each thread also loads its 32 values of W and 16 bytes of the
//      new K / V rows into registers;
//   2. the G query rows and the key row are hashed with the library-wide projection order (Eq. 2);
//   3. every slot's Hamming distance to the query codes (Eq. 5) is taken from shared memory, scores are stored,
//      and the arg-max (Eq. 6, lowest index on ties) is a packed-key redux.sync + one block barrier;
//   4. the victim slot's K, V, code and position are overwritten in place.
#pragma once
#include <type_traits>

#include "common.cuh"

namespace he {

constexpr int kMaxBudgetVals = 1024;  // budgets carried in the kernel parameters (4 KB)

struct DecodeArgs {
  he_config cfg;
  he_cache ca;
  const void* q;
  const void* k;
  const void* v;
  int32_t* victim_out;
  int32_t* evicted_pos_out;
  uint32_t* qcodes_out;
  const uint32_t* new_codes;               // PRE kernels: [B*Hkv*G + B*Hkv, Wd] codes of this step's q rows, then k rows
  int n_budget_vals;                       // > 0: budgets are in budget_vals (copied from he_cache.budget_host)
  int n_sched;                             // > 0: sched lists the sequences by budget, largest first (sequence << 21 | budget)
  int32_t budget_vals[kMaxBudgetVals];
  uint32_t sched[kMaxBudgetVals];
};

constexpr int kVecsPerThread = 8;  // 16-byte code vectors per thread (the host picks the block size accordingly)
constexpr int kRowBatch = 5;  // rows hashed per pass (G = 4 queries + the key in one pass)

// -(float)D for a small non-negative integer D without an int->float conversion (a quarter-rate instruction):
// the bit pattern 0x4B000000 + D is the float 2^23 + D.
__device__ __forceinline__ float neg_small_int(int D) { return 8388608.0f - __uint_as_float(0x4B000000u + (uint32_t)D); }

// PRE = true (large batches): the codes of the step's new rows were written to a.new_codes by the bulk projection
// kernels launched just before this one in the stream, which themselves started only after everything earlier had
// finished. So the cache state and the step's k / v rows may be read BEFORE griddepcontrol.wait here; only new_codes
// is read after it.
//
// PACKED = true (HE_FLAG_PACKED_CODES with fewer bytes per slot than the word layout; WORDS = 1): the table holds
// cb = ceil(b/8) bytes per slot, 1 to 3. A thread takes four consecutive slots (cb words) at a time, widens each code
// to a word in registers and scores it like a word-layout slot.
template <int WORDS, int GT, int NT, bool PRE, bool PACKED = false>
__global__ void __launch_bounds__(NT, (NT <= 256 ? (PRE ? 6 : 4) : 1)) decode_step_kernel(const DecodeArgs a) {
  static_assert(!PACKED || WORDS == 1, "packed tables hold codes of at most 24 bits");
  constexpr int SPV = 4 / WORDS;  // slots per 16-byte vector
  constexpr int BP = 32 * WORDS;
  constexpr bool kGroupedCopy = WORDS == 2;
  using Ctx = QueryCtx<WORDS, GT>;
  extern __shared__ __align__(16) uint32_t dsm[];  // the unit's code words
  // staging of the rows to hash and of the partial sums: not needed when the codes come pre-hashed
  __shared__ __align__(16) float xs[PRE ? 1 : kRowBatch][PRE ? 4 : kMaxDim];
  __shared__ float part[PRE ? 1 : kMaxDim / kChunk][PRE ? 1 : kRowBatch][PRE ? 1 : BP];
  __shared__ __align__(16) uint32_t codes_s[(kMaxGroup + 1) * WORDS];  // rows 0..G-1: query codes, row G: key code
  __shared__ uint32_t wbest[2][32];

  griddep_launch_dependents();
  const he_config& cfg = a.cfg;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int s = blockIdx.y;
  const int unit = s * cfg.n_kv_heads + blockIdx.x;
  const int d = cfg.head_dim, b = cfg.hash_bits, G = cfg.group_size, es = esize_of(cfg.dtype);
  const int Cmax = cfg.max_budget;

  // Hashing work item = (chunk of 32 channels, bit). In the dense shape (b = 32 or 64, whole chunks, one item per
  // thread, one pass of rows) the thread's 32 values of W are fetched right away: W never changes while a cache
  // is in use, so this read may overlap the tail of the previous kernel of the stream.
  const int R = G + 1;
  const int nch = (d + kChunk - 1) / kChunk;
  const int nitems = nch * BP;
  const int cpr = d * es / 16;  // 16-byte chunks per row
  const bool dense = !PRE && nitems <= NT && R <= kRowBatch && cpr <= 32;  // one item per thread, one pass, one chunk per lane
  float wreg[kChunk];
  if (dense && tid < nitems) {
    const int c0 = (tid / BP) * kChunk, bi = tid % BP;
    if (b == BP && d % kChunk == 0) {  // b = 32 or 64 and whole chunks: constant strides, no edge tests
      const float* wp = a.ca.W + c0 * BP + bi;
#pragma unroll
      for (int cc = 0; cc < kChunk; ++cc) wreg[cc] = __ldg(wp + cc * BP);
    } else {  // columns beyond b and channels beyond d count as zeros
      const int clen = bi < b ? min(kChunk, d - c0) : 0;
      const float* wp = a.ca.W + c0 * b + bi;
#pragma unroll
      for (int cc = 0; cc < kChunk; ++cc) wreg[cc] = cc < clen ? __ldg(wp + cc * b) : 0.f;
    }
  }

  if (!PRE) griddep_wait();
  // The rows to hash are requested before the code table: they head the dependency chain, the table only has to
  // be there when hashing is done.
  uint4 xraw = make_uint4(0u, 0u, 0u, 0u);
  const bool stages = dense && warp < R && lane < cpr;
  if (stages) {
    const char* src = warp < G ? static_cast<const char*>(a.q) + ((size_t)unit * G + warp) * d * es
                               : static_cast<const char*>(a.k) + (size_t)unit * d * es;
    xraw = __ldg(reinterpret_cast<const uint4*>(src) + lane);
  }
  // the new K and V rows, 16 bytes per thread, kept until the victim is known
  uint4 rowreg = make_uint4(0u, 0u, 0u, 0u);
  if (tid < 2 * cpr) {
    const bool is_k = tid < cpr;
    const char* src = static_cast<const char*>(is_k ? a.k : a.v) + (size_t)unit * d * es;
    rowreg = __ldg(reinterpret_cast<const uint4*>(src) + (is_k ? tid : tid - cpr));
  }
  const int C = clamp_budget(a.n_budget_vals > 0 ? a.budget_vals[s] : a.ca.budget[s], Cmax);
  const int fill = a.ca.fill[unit];
  const int t = a.ca.next_pos[unit];

  // (1) code words -> shared memory, asynchronously. The copy is sized by the budget alone: if the unit turns out
  // to be still filling (fill < C) the copied words are simply not used.
  const int cb = PACKED ? (b + 7) >> 3 : 0;
  const int nvec = PACKED ? (C * cb + 15) / 16 : (C * WORDS + 3) / 4;
  {
    const uint4* cvec = PACKED ? reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(a.ca.codes) + (size_t)unit * Cmax * cb)
                               : reinterpret_cast<const uint4*>(a.ca.codes + (size_t)unit * Cmax * WORDS);
    // Two-word codes (b > 32): one commit group per vector of this thread; the scan waits for them one by one and
    // reads only what this thread copied itself, so it overlaps the rest of the transfer. Measured on B200 this is
    // 6 % faster per call at b = 64 but slower at b <= 32 (larger unrolled scan body), where a single group is used.
    if (kGroupedCopy) {
#pragma unroll
      for (int i = 0; i < kVecsPerThread; ++i) {
        const int vi = i * NT + tid;
        if (vi < nvec) cp_async16(dsm + 4 * vi, cvec + vi);
        cp_async_commit();
      }
    } else {
      for (int vi = tid; vi < nvec; vi += NT) cp_async16(dsm + 4 * vi, cvec + vi);
      cp_async_commit();
    }
  }

  // (2) hash the G query rows and the key row (Eq. 2): one fmaf chain per row and work item, partial sums combined
  // through shared memory in chunk order.
  if (PRE) {
    griddep_wait();
    const size_t nq = (size_t)gridDim.x * gridDim.y * G;
    if (tid < G * WORDS) codes_s[tid] = __ldcg(a.new_codes + (size_t)unit * G * WORDS + tid);
    else if (tid < R * WORDS) codes_s[tid] = __ldcg(a.new_codes + (nq + unit) * WORDS + (tid - G * WORDS));
  }
  auto stage_rows = [&](int r0) {  // warp r stages row r0 + r as fp32
    if (warp < kRowBatch) {
      const int row = r0 + warp;
      if (row < R) {
        const char* src = row < G ? static_cast<const char*>(a.q) + ((size_t)unit * G + row) * d * es
                                  : static_cast<const char*>(a.k) + (size_t)unit * d * es;
        for (int ch = lane; ch < cpr; ch += 32) stage_chunk(xs[warp], src, ch, cfg.dtype);
      } else {
        for (int c = lane; c < d; c += 32) xs[warp][c] = 0.f;
      }
    }
  };
  auto combine = [&](int r0) {  // partial sums -> sign bits, one ballot per (row, code word)
    for (int task = warp; task < kRowBatch * WORDS; task += NT / 32) {
      const int r = task / WORDS, w = task % WORDS;
      float tot = 0.f;
      for (int q2 = 0; q2 < nch; ++q2) tot += part[q2][r][w * 32 + lane];
      const uint32_t word = __ballot_sync(0xFFFFFFFFu, tot >= 0.f) & word_mask(b, w);
      if (lane == 0 && r0 + r < R) codes_s[(r0 + r) * WORDS + w] = word;
    }
  };
  if (PRE) {
    // nothing to hash in this kernel
  } else if (dense) {
    const bool active = tid < nitems;
    const int qd = tid / BP, bi = tid % BP;
    if (stages) store_chunk(xs[warp], xraw, lane, cfg.dtype);
    if (warp < kRowBatch)  // zeros for absent rows and for the channels that pad the last chunk
      for (int c = (warp < R ? d : 0) + lane; c < nch * kChunk; c += 32) xs[warp][c] = 0.f;
    __syncthreads();
    if (active) {
      float acc[kRowBatch];
#pragma unroll
      for (int r = 0; r < kRowBatch; ++r) acc[r] = 0.f;
      const float* xb = &xs[0][qd * kChunk];
#pragma unroll
      for (int cc = 0; cc < kChunk; cc += 4) {
#pragma unroll
        for (int r = 0; r < kRowBatch; ++r) {
          const float4 xv = *reinterpret_cast<const float4*>(xb + r * kMaxDim + cc);
          acc[r] = fmaf(xv.x, wreg[cc], acc[r]);
          acc[r] = fmaf(xv.y, wreg[cc + 1], acc[r]);
          acc[r] = fmaf(xv.z, wreg[cc + 2], acc[r]);
          acc[r] = fmaf(xv.w, wreg[cc + 3], acc[r]);
        }
      }
#pragma unroll
      for (int r = 0; r < kRowBatch; ++r) part[qd][r][bi] = acc[r];
    }
    __syncthreads();
    combine(0);
  } else {
    for (int r0 = 0; r0 < R; r0 += kRowBatch) {
      if (r0 > 0) __syncthreads();
      stage_rows(r0);
      __syncthreads();
      for (int item = tid; item < nitems; item += NT) {
        const int qd = item / BP, bi = item % BP, c0 = qd * kChunk;
        const int clen = min(kChunk, d - c0);
        float acc[kRowBatch];
#pragma unroll
        for (int r = 0; r < kRowBatch; ++r) acc[r] = 0.f;
        if (bi < b) {
          for (int cc = 0; cc < clen; cc += 4) {  // d is a multiple of 8
            float wv[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) wv[k] = __ldg(a.ca.W + (c0 + cc + k) * b + bi);
#pragma unroll
            for (int r = 0; r < kRowBatch; ++r) {
              const float4 xv = *reinterpret_cast<const float4*>(&xs[r][c0 + cc]);
              acc[r] = fmaf(xv.x, wv[0], acc[r]);
              acc[r] = fmaf(xv.y, wv[1], acc[r]);
              acc[r] = fmaf(xv.z, wv[2], acc[r]);
              acc[r] = fmaf(xv.w, wv[3], acc[r]);
            }
          }
        }
#pragma unroll
        for (int r = 0; r < kRowBatch; ++r) part[qd][r][bi] = acc[r];
      }
      __syncthreads();
      combine(r0);
    }
  }
  if (!kGroupedCopy) cp_async_wait_all();  // this thread's code copies have landed
  __syncthreads();                         // the codes of the new rows (and, ungrouped, the table) are in shared memory
  if (a.qcodes_out != nullptr && tid < G * WORDS) a.qcodes_out[(size_t)unit * G * WORDS + tid] = codes_s[tid];

  // (3) Eq. 5 / Eq. 6
  const bool evict = C >= 1 && fill >= C;
  int slot = fill;
  if (evict) {
    Ctx ctx;
    if (GT == 4) {  // build the bit-plane record in registers
      uint32_t rec[Ctx::kRecWords];
      Ctx::build(rec, codes_s, G);
      ctx.load(rec, G);
    } else {
      ctx.load(codes_s, G);
    }
    const bool prot = cfg.n_sink > 0 || cfg.n_recent > 0;
    const bool write_scores = (cfg.flags & HE_FLAG_WRITE_SCORES) != 0;
    float* sc = a.ca.scores + (size_t)unit * Cmax;
    const int32_t* pp = a.ca.pos + (size_t)unit * Cmax;
    constexpr uint32_t kKeyBase = (1u << kKeyIdxBits) + kKeyIdxMask;  // key = (rank << 20) + kKeyBase - slot
    uint32_t best_all = 0u, best_el = 0u;
    // one pass over the unit's vectors; PROT and SCORES are compile-time in each instantiation of the loop body
    auto scan = [&](auto prot_c, auto scores_c) {
      constexpr bool PROT = decltype(prot_c)::value, SCORES = decltype(scores_c)::value;
#pragma unroll(kGroupedCopy ? kVecsPerThread : 2)
      for (int i = 0; i < kVecsPerThread; ++i) {
        if (!kGroupedCopy && i * NT >= nvec) break;
        if (kGroupedCopy) cp_async_wait_pending(kVecsPerThread - 1 - i);  // this thread's i-th vector has landed
        const int vi = i * NT + tid;
        if (vi >= nvec) continue;
        const uint4 cvv = *reinterpret_cast<const uint4*>(dsm + 4 * vi);
        const uint32_t wds[4] = {cvv.x, cvv.y, cvv.z, cvv.w};
        const int j0 = vi * SPV;
        int rk[SPV];
#pragma unroll
        for (int e = 0; e < SPV; ++e) {
          uint32_t h[WORDS];
#pragma unroll
          for (int w = 0; w < WORDS; ++w) h[w] = wds[e * WORDS + w];
          rk[e] = ctx.rank(h);
        }
        if (j0 + SPV <= C) {  // every vector but possibly a unit's last one
#pragma unroll
          for (int e = 0; e < SPV; ++e) {
            const uint32_t key = ((uint32_t)rk[e] << kKeyIdxBits) + (kKeyBase - (uint32_t)(j0 + e));
            best_all = max(best_all, key);
            if (PROT) {
              const int p = __ldg(pp + j0 + e);
              if (p >= cfg.n_sink && p < t - cfg.n_recent) best_el = max(best_el, key);
            }
          }
          if (SCORES) {
            if (SPV == 4)
              *reinterpret_cast<float4*>(sc + j0) =
                  make_float4(neg_small_int(ctx.dist(rk[0])), neg_small_int(ctx.dist(rk[1])),
                              neg_small_int(ctx.dist(rk[SPV > 2 ? 2 : 0])), neg_small_int(ctx.dist(rk[SPV > 3 ? 3 : 0])));
            else
              *reinterpret_cast<float2*>(sc + j0) = make_float2(neg_small_int(ctx.dist(rk[0])), neg_small_int(ctx.dist(rk[1])));
          }
        } else {
#pragma unroll
          for (int e = 0; e < SPV; ++e)
            if (j0 + e < C) {
              const uint32_t key = ((uint32_t)rk[e] << kKeyIdxBits) + (kKeyBase - (uint32_t)(j0 + e));
              best_all = max(best_all, key);
              if (PROT) {
                const int p = __ldg(pp + j0 + e);
                if (p >= cfg.n_sink && p < t - cfg.n_recent) best_el = max(best_el, key);
              }
              if (SCORES) sc[j0 + e] = neg_small_int(ctx.dist(rk[e]));
            }
        }
      }
    };
    using T = std::true_type;
    using F = std::false_type;
    // packed table: CB bytes per slot; like a word-layout vector, a group is four consecutive slots (CB words)
    auto scan_packed = [&](auto cb_c, auto prot_c, auto scores_c) {
      constexpr int CB = decltype(cb_c)::value;
      constexpr bool PROT = decltype(prot_c)::value, SCORES = decltype(scores_c)::value;
      const int ngroups = (C + 3) / 4;
#pragma unroll 2
      for (int gi = tid; gi < ngroups; gi += NT) {
        uint32_t wd[CB];
        if (CB == 2) {
          const uint2 x = *reinterpret_cast<const uint2*>(dsm + gi * CB);
          wd[0] = x.x, wd[CB - 1] = x.y;
        } else {
#pragma unroll
          for (int i = 0; i < CB; ++i) wd[i] = dsm[gi * CB + i];
        }
        const int j0 = gi * 4;
        const bool whole = j0 + 4 <= C;
        int rk[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          constexpr int kBits = 8 * CB;
          const int o = e * kBits;  // bit offset of the slot's code inside the group
          uint32_t h[WORDS] = {};  // WORDS is 1 wherever this runs
          if (CB == 3) h[0] = __funnelshift_r(wd[o >> 5], wd[(o >> 5) + 1 < CB ? (o >> 5) + 1 : CB - 1], o & 31) & 0xFFFFFFu;
          else h[0] = (wd[o >> 5] >> (o & 31)) & ((1u << kBits) - 1u);
          rk[e] = ctx.rank(h);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int j = j0 + e;
          if (whole || j < C) {
            const uint32_t key = ((uint32_t)rk[e] << kKeyIdxBits) + (kKeyBase - (uint32_t)j);
            best_all = max(best_all, key);
            if (PROT) {
              const int p = __ldg(pp + j);
              if (p >= cfg.n_sink && p < t - cfg.n_recent) best_el = max(best_el, key);
            }
            if (SCORES && !whole) sc[j] = neg_small_int(ctx.dist(rk[e]));
          }
        }
        if (SCORES && whole)
          *reinterpret_cast<float4*>(sc + j0) = make_float4(neg_small_int(ctx.dist(rk[0])), neg_small_int(ctx.dist(rk[1])),
                                                            neg_small_int(ctx.dist(rk[2])), neg_small_int(ctx.dist(rk[3])));
      }
    };
    auto scan_packed_cb = [&](auto prot_c, auto scores_c) {
      if (cb == 1) scan_packed(std::integral_constant<int, 1>{}, prot_c, scores_c);
      else if (cb == 2) scan_packed(std::integral_constant<int, 2>{}, prot_c, scores_c);
      else scan_packed(std::integral_constant<int, 3>{}, prot_c, scores_c);
    };
    if constexpr (PACKED) {
      if (prot) {
        if (write_scores) scan_packed_cb(T{}, T{}); else scan_packed_cb(T{}, F{});
      } else {
        if (write_scores) scan_packed_cb(F{}, T{}); else scan_packed_cb(F{}, F{});
      }
    } else if (prot) {
      if (write_scores) scan(T{}, T{}); else scan(T{}, F{});
    } else {
      if (write_scores) scan(F{}, T{}); else scan(F{}, F{});
    }
    uint32_t fin = block_max_key(best_all, wbest[0], lane, warp, NT / 32);
    if (prot) {
      const uint32_t fin_el = block_max_key(best_el, wbest[1], lane, warp, NT / 32);
      if (fin_el != 0u) fin = fin_el;
    }
    slot = (int)(kKeyIdxMask - (fin & kKeyIdxMask));
  }

  if (!evict) cp_async_wait_all();  // a unit that is still filling never looked at the copied table
  if (C < 1 || !HE_IN_RANGE(slot, C)) {  // a unit without a budget holds nothing: report it and leave the state alone
    if (tid == 0) {
      a.victim_out[unit] = -1;
      if (a.evicted_pos_out != nullptr) a.evicted_pos_out[unit] = -1;
    }
    return;
  }
  // (4) Algorithm 1 lines 2-5: the slot takes the new token's K, V, code and position
  const size_t slot_idx = (size_t)unit * Cmax + slot;
  if (tid < 2 * cpr) {
    const bool is_k = tid < cpr;
    char* dst = static_cast<char*>(is_k ? a.ca.k_cache : a.ca.v_cache) + slot_idx * d * es;
    reinterpret_cast<uint4*>(dst)[is_k ? tid : tid - cpr] = rowreg;
  }
  if (tid == NT - 1) {
    int ev = -1;
    if (evict && a.evicted_pos_out != nullptr) ev = a.ca.pos[slot_idx];
    a.ca.pos[slot_idx] = t;
    if (PACKED) {
      for (int i = 0; i < cb; ++i) reinterpret_cast<uint8_t*>(a.ca.codes)[slot_idx * cb + i] = (uint8_t)(codes_s[G] >> (8 * i));
    } else {
#pragma unroll
      for (int w = 0; w < WORDS; ++w) a.ca.codes[slot_idx * WORDS + w] = codes_s[G * WORDS + w];
    }
    if (!evict) {
      a.ca.scores[slot_idx] = 0.f;
      a.ca.fill[unit] = fill + 1;
    }
    a.ca.next_pos[unit] = t + 1;
    a.victim_out[unit] = slot;
    if (a.evicted_pos_out != nullptr) a.evicted_pos_out[unit] = ev;
  }
}

}  // namespace he
