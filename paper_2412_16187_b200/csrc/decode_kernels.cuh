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
#include "common.cuh"

namespace he {

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

constexpr int kRowBatch = 5;  // rows hashed per pass (G = 4 queries + the key in one pass)

template <int WORDS, int GT, int NT>
__global__ void __launch_bounds__(NT, (NT <= 256 ? 4 : 1)) decode_step_kernel(const DecodeArgs a) {
  constexpr int SPV = 4 / WORDS;  // slots per 16-byte vector
  constexpr int BP = 32 * WORDS;
  extern __shared__ __align__(16) uint32_t dsm[];  // the unit's code words
  __shared__ __align__(16) float xs[kRowBatch][kMaxDim];
  __shared__ float part[kMaxDim / kChunk][kRowBatch][BP];
  __shared__ __align__(16) uint32_t codes_s[(kMaxGroup + 1) * WORDS];  // rows 0..G-1: query codes, row G: key code
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

  // (1) code words -> shared memory, asynchronously
  const int nvec = evict ? (C * WORDS + 3) / 4 : 0;
  {
    const uint4* cvec = reinterpret_cast<const uint4*>(a.ca.codes + unit * Cmax * WORDS);
    for (int vi = tid; vi < nvec; vi += NT) cp_async16(dsm + 4 * vi, cvec + vi);
    cp_async_commit();
  }
  // this thread's slice of W for the projection: item = (chunk qd of the channels, bit bi); when there are no more
  // items than threads (every shape with d <= 128), the 32 values of W are loaded once, before anything is waited on
  const int nch = (d + kChunk - 1) / kChunk;
  const int nitems = nch * BP;
  const bool w_resident = nitems <= NT;
  float wreg[kChunk];
  auto load_w = [&](int item) {
    const int c0 = (item / BP) * kChunk, bi = item % BP;
#pragma unroll
    for (int cc = 0; cc < kChunk; ++cc)
      wreg[cc] = (item < nitems && bi < b && c0 + cc < d) ? __ldg(a.ca.W + (long long)(c0 + cc) * b + bi) : 0.f;
  };
  load_w(tid);
  // the new K and V rows, 16 bytes per thread, kept until the victim is known
  const int cpr = d * es / 16;
  uint4 rowreg = make_uint4(0u, 0u, 0u, 0u);
  if (tid < 2 * cpr) {
    const char* src = static_cast<const char*>(tid < cpr ? a.k : a.v) + unit * d * es;
    rowreg = __ldg(reinterpret_cast<const uint4*>(src) + (tid % cpr));
  }

  // (2) hash the G query rows and the key row (Eq. 2)
  const int R = G + 1;
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
    for (int item = tid; item < nitems; item += NT) {
      if (!w_resident) load_w(item);
      const int qd = item / BP, bi = item % BP;
      float acc[kRowBatch];
#pragma unroll
      for (int r = 0; r < kRowBatch; ++r) acc[r] = 0.f;
      const int c0 = qd * kChunk;
#pragma unroll
      for (int cc = 0; cc < kChunk; cc += 4) {
        if (c0 + cc < d) {  // d is a multiple of 8, so a group of four channels is all in or all out
#pragma unroll
          for (int r = 0; r < kRowBatch; ++r) {
            const float4 xv = *reinterpret_cast<const float4*>(&xs[r][c0 + cc]);
            acc[r] = fmaf(xv.x, wreg[cc], acc[r]);
            acc[r] = fmaf(xv.y, wreg[cc + 1], acc[r]);
            acc[r] = fmaf(xv.z, wreg[cc + 2], acc[r]);
            acc[r] = fmaf(xv.w, wreg[cc + 3], acc[r]);
          }
        }
      }
#pragma unroll
      for (int r = 0; r < kRowBatch; ++r) part[qd][r][bi] = acc[r];
    }
    __syncthreads();
    for (int task = warp; task < kRowBatch * WORDS; task += NT / 32) {
      const int r = task / WORDS, w = task % WORDS;
      float tot = 0.f;
      for (int q2 = 0; q2 < nch; ++q2) tot += part[q2][r][w * 32 + lane];
      const uint32_t word = __ballot_sync(0xFFFFFFFFu, tot >= 0.f) & word_mask(b, w);
      if (lane == 0 && r0 + r < R) codes_s[(r0 + r) * WORDS + w] = word;
    }
    cp_async_wait_all();  // (no-op after the first pass) this thread's code copies have landed
    __syncthreads();
  }
  if (a.qcodes_out != nullptr && tid < G * WORDS) a.qcodes_out[unit * G * WORDS + tid] = codes_s[tid];

  // (3) Eq. 5 / Eq. 6
  int slot = fill;
  if (evict) {
    QueryCtx<WORDS, GT> ctx;
    if (GT == 4) {  // build the bit-plane record in registers
      uint32_t rec[QueryCtx<WORDS, GT>::kRecWords];
      QueryCtx<WORDS, GT>::build(rec, codes_s, G);
      ctx.load(rec, G);
    } else {
      ctx.load(codes_s, G);
    }
    const bool prot = cfg.n_sink > 0 || cfg.n_recent > 0;
    const bool write_scores = (cfg.flags & HE_FLAG_WRITE_SCORES) != 0;
    float* sc = a.ca.scores + unit * Cmax;
    const int32_t* pp = a.ca.pos + unit * Cmax;
    uint32_t best_all = 0u, best_el = 0u;
#pragma unroll 2
    for (int vi = tid; vi < nvec; vi += NT) {
      const uint4 cvv = *reinterpret_cast<const uint4*>(dsm + 4 * vi);
      const uint32_t wds[4] = {cvv.x, cvv.y, cvv.z, cvv.w};
      const int j0 = vi * SPV;
      float sv[SPV];
#pragma unroll
      for (int e = 0; e < SPV; ++e) {
        const int j = j0 + e;
        uint32_t h[WORDS];
#pragma unroll
        for (int w = 0; w < WORDS; ++w) h[w] = wds[e * WORDS + w];
        const int rk = ctx.rank(h);
        sv[e] = -(float)ctx.dist(rk);
        if (j < C) {
          const uint32_t key = ((uint32_t)(rk + 1) << kKeyIdxBits) | (kKeyIdxMask - (uint32_t)j);
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
    uint32_t fin = block_max_key(best_all, wbest[0], lane, warp, NT / 32);
    if (prot) {
      const uint32_t fin_el = block_max_key(best_el, wbest[1], lane, warp, NT / 32);
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

}  // namespace he
