// he_attend: Eq. 1 over the compressed cache (Algorithm 1 line 6), the step that follows the eviction:
//   out[g] = sum_j softmax_j(q_g . K_j / sqrt(d)) V_j   over the valid slots of the query head's KV unit.
// All G query heads of a group are served together, so K and V are read once for the group. Each warp walks its
// own slots with an online softmax (running maximum, running sum, unnormalised output) and the partial results are
// merged through shared memory at the end. HBM-bound by design: 2 * C * d * e bytes per unit.
//
//   attend_bf16_kernel     bf16, d = 128, G <= 8: 16 slots at a time, Q K^T and P V as warp-level m16n8k16 MMAs fed
//                          straight from registers (bf16 products are exact, fp32 accumulation, P as hi + lo bf16);
//                          a cluster of up to 8 CTAs shares a unit when there are few units.
//   attend_generic_kernel  any supported dtype / d: one slot at a time, dot products by warp shuffles.
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"

namespace he {

struct AttendArgs {
  he_config cfg;
  he_cache ca;
  const void* q;  // [B, Hkv*G, d]
  float* out;     // [B, Hkv*G, d] fp32
};

constexpr int kAttendThreads = 256;
constexpr int kAttendWarps = kAttendThreads / 32;
constexpr float kLog2e = 1.4426950408889634f;

// Merge of the per-warp partial results (m = running max in log2 units, l = running sum, o = unnormalised output).
// part_ml: [warps][G][2], part_o: [warps][G][d]. Every thread writes some of the G * d outputs.
__device__ __forceinline__ void attend_merge(const float* part_ml, const float* part_o, int G, int d, float* out_unit) {
  for (int idx = threadIdx.x; idx < G * d; idx += kAttendThreads) {
    const int g = idx / d, c = idx % d;
    float M = -INFINITY;
    for (int w = 0; w < kAttendWarps; ++w) M = fmaxf(M, part_ml[(w * G + g) * 2]);
    float L = 0.f, O = 0.f;
    for (int w = 0; w < kAttendWarps; ++w) {
      const float m = part_ml[(w * G + g) * 2];
      const float f = m == -INFINITY ? 0.f : exp2f(m - M);
      L += part_ml[(w * G + g) * 2 + 1] * f;
      O += part_o[(w * G + g) * d + c] * f;
    }
    out_unit[idx] = L > 0.f ? O / L : 0.f;
  }
}

// Two-level merge for a cluster of S CTAs on one unit: each CTA folds its warps into (cta_ml, cta_o) in its own
// shared memory, then every CTA combines the S partial results for its share of the G * d outputs, reading the
// other CTAs' shared memory. The last cluster barrier keeps every CTA's shared memory alive until all have read it.
__device__ __forceinline__ void attend_merge_cluster(const float* part_ml, const float* part_o, float* cta_ml, float* cta_o,
                                                     int G, int d, int S, int rank, float* out_unit) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  for (int idx = threadIdx.x; idx < G * d; idx += kAttendThreads) {
    const int g = idx / d, c = idx % d;
    float M = -INFINITY;
    for (int w = 0; w < kAttendWarps; ++w) M = fmaxf(M, part_ml[(w * G + g) * 2]);
    float L = 0.f, O = 0.f;
    for (int w = 0; w < kAttendWarps; ++w) {
      const float m = part_ml[(w * G + g) * 2];
      const float f = m == -INFINITY ? 0.f : exp2f(m - M);
      L += part_ml[(w * G + g) * 2 + 1] * f;
      O += part_o[(w * G + g) * d + c] * f;
    }
    if (c == 0) cta_ml[g * 2] = M, cta_ml[g * 2 + 1] = L;
    cta_o[idx] = O;
  }
  cluster.sync();
  const int total = G * d, share = (total + S - 1) / S;
  const int hi = min(total, (rank + 1) * share);
  for (int idx = rank * share + threadIdx.x; idx < hi; idx += kAttendThreads) {
    const int g = idx / d;
    float M = -INFINITY;
    for (int r = 0; r < S; ++r) M = fmaxf(M, cluster.map_shared_rank(cta_ml, r)[g * 2]);
    float L = 0.f, O = 0.f;
    for (int r = 0; r < S; ++r) {
      const float* ml = cluster.map_shared_rank(cta_ml, r);
      const float m = ml[g * 2];
      const float f = m == -INFINITY ? 0.f : exp2f(m - M);
      L += ml[g * 2 + 1] * f;
      O += cluster.map_shared_rank(cta_o, r)[idx] * f;
    }
    out_unit[idx] = L > 0.f ? O / L : 0.f;
  }
  cluster.sync();
}

// ------------------------------------------------------------------------------------------------ bf16, d = 128
//
// A warp takes 16 slots at a time. Scores: S[head][slot] = Q K^T as m16n8k16 MMAs with M = query heads (rows 0..7
// used), N = 8 slots, K = 16 channels. A dot product does not depend on the order of its terms, so the 16 "logical"
// channels of MMA step s are chosen to suit 16-byte loads: lane (gid, tig) reads chunks tig, tig+4, tig+8, tig+12
// (8 channels each) of row gid, and chunk tig+4c feeds steps 2c (first two registers) and 2c+1 (last two); the
// query fragment is loaded the same way, so both operands agree on the permutation.
// Output: O[head][channel] += P V with M = heads, K = 16 slots, N = 8 channels. The score tile's accumulator layout
// is already the A-fragment layout of P (head gid, slots 2tig, 2tig+1 [+8]). P is split into two bf16 terms
// (p = hi + lo + O(2^-18 p)): hi in rows 0..7, lo in rows 8..15 of the same MMA, summed at the end, so that the
// rows a group of <= 8 heads leaves empty carry the low-order term. The B fragment wants pairs of slots per
// channel: lane (gid, tig) holds slots 2tig, 2tig+1, 2tig+8, 2tig+9 and chunks gid, gid+8 of each, and a byte
// permute pairs the two slots' values of one channel. Output tile t = 8h + e of lane column n is channel
// (n + 8h) * 8 + e.

__device__ __forceinline__ void mma_bf16_m16n8k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                  uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// (hi, lo) bf16 pairs of two fp32 values: hi = round-to-nearest bf16, lo = bf16 of the exact remainder.
// The first value goes to the low half (the lower k index of the fragment).
__device__ __forceinline__ void split_pair(float x, float y, uint32_t& hi, uint32_t& lo) {
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(hi) : "f"(y), "f"(x));
  const float xr = x - __uint_as_float(hi << 16), yr = y - __uint_as_float(hi & 0xFFFF0000u);
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(lo) : "f"(yr), "f"(xr));
}

__device__ __forceinline__ uint4 ldg_stream16(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// Grid (Hkv * S, B) in clusters of S CTAs along x: the S CTAs of a cluster share one unit's slots (16-slot groups
// dealt round-robin over the S * 8 warps), each merges its own warps, and the cluster merges the S partial results
// through distributed shared memory, so a call with few units still fills the GPU without any scratch in HBM.
// Dynamic shared memory: part_ml [warps][G][2], part_o [warps][G][d], cta_ml [G][2], cta_o [G][d] floats.
__global__ void __launch_bounds__(kAttendThreads, 1) attend_bf16_kernel(const AttendArgs a, const int S) {
  extern __shared__ __align__(16) float asm_[];
  constexpr int d = 128;
  const he_config& cfg = a.cfg;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, gid = lane >> 2, tig = lane & 3;
  const int rank = blockIdx.x % S;
  const int unit = blockIdx.y * cfg.n_kv_heads + blockIdx.x / S;
  const int G = cfg.group_size;
  const int fill = a.ca.fill[unit];
  float* part_ml = asm_;
  float* part_o = part_ml + kAttendWarps * G * 2;
  float* cta_ml = part_o + kAttendWarps * G * d;
  float* cta_o = cta_ml + G * 2;
  const uint4* Kb = static_cast<const uint4*>(a.ca.k_cache) + (size_t)unit * cfg.max_budget * (d / 8);
  const uint4* Vb = static_cast<const uint4*>(a.ca.v_cache) + (size_t)unit * cfg.max_budget * (d / 8);

  uint32_t qf[8][2];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    uint4 t = make_uint4(0u, 0u, 0u, 0u);
    if (gid < G) t = static_cast<const uint4*>(a.q)[((size_t)unit * G + gid) * (d / 8) + tig + 4 * c];
    qf[2 * c][0] = t.x, qf[2 * c][1] = t.y, qf[2 * c + 1][0] = t.z, qf[2 * c + 1][1] = t.w;
  }
  const float scale = rsqrtf((float)d) * kLog2e;
  const int last = fill - 1;
  // Rows past the fill level are read from the last valid row (finite data) and weighted by zero.
  auto load_k = [&](int g0, uint4 (&kb)[2][4]) {
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const uint4* row = Kb + (size_t)min(g0 + gid + 8 * r, last) * (d / 8);
#pragma unroll
      for (int c = 0; c < 4; ++c) kb[r][c] = ldg_stream16(row + tig + 4 * c);
    }
  };
  auto load_v = [&](int g0, uint4 (&vb)[4][2]) {
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const uint4* row = Vb + (size_t)min(g0 + 2 * tig + (s & 1) + 8 * (s >> 1), last) * (d / 8);
      vb[s][0] = ldg_stream16(row + gid);
      vb[s][1] = ldg_stream16(row + gid + 8);
    }
  };
  float m = -INFINITY, l = 0.f;
  float o[16][4];
#pragma unroll
  for (int t = 0; t < 16; ++t) o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f;
  uint4 kc[2][4], vc[4][2], kn[2][4], vn[4][2];
  const int stride = 16 * kAttendWarps * S;
  int g0 = 16 * (warp * S + rank);
  if (g0 < fill) {
    load_k(g0, kc);
    load_v(g0, vc);
  }
  for (; g0 < fill; g0 += stride) {
    const bool more = g0 + stride < fill;
    if (more) load_k(g0 + stride, kn);
    float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      mma_bf16_m16n8k16(s0, qf[2 * c][0], 0u, qf[2 * c][1], 0u, kc[0][c].x, kc[0][c].y);
      mma_bf16_m16n8k16(s1, qf[2 * c][0], 0u, qf[2 * c][1], 0u, kc[1][c].x, kc[1][c].y);
      mma_bf16_m16n8k16(s0, qf[2 * c + 1][0], 0u, qf[2 * c + 1][1], 0u, kc[0][c].z, kc[0][c].w);
      mma_bf16_m16n8k16(s1, qf[2 * c + 1][0], 0u, qf[2 * c + 1][1], 0u, kc[1][c].z, kc[1][c].w);
    }
    // This lane: head gid, slots g0 + 2tig, + 1, + 8, + 9.
    const int j = g0 + 2 * tig;
    const float x0 = j < fill ? s0[0] * scale : -INFINITY, x1 = j + 1 < fill ? s0[1] * scale : -INFINITY;
    const float x2 = j + 8 < fill ? s1[0] * scale : -INFINITY, x3 = j + 9 < fill ? s1[1] * scale : -INFINITY;
    float gm = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
    gm = fmaxf(gm, __shfl_xor_sync(0xFFFFFFFFu, gm, 1));
    gm = fmaxf(gm, __shfl_xor_sync(0xFFFFFFFFu, gm, 2));  // finite: slot g0 is valid
    const float mn = fmaxf(m, gm);
    const float corr = exp2f(m - mn);
    const float p0 = exp2f(x0 - mn), p1 = exp2f(x1 - mn), p2 = exp2f(x2 - mn), p3 = exp2f(x3 - mn);
    l = l * corr + ((p0 + p1) + (p2 + p3));
    m = mn;
    uint32_t a0, a1, a2, a3;
    split_pair(p0, p1, a0, a1);
    split_pair(p2, p3, a2, a3);
    if (more) load_v(g0 + stride, vn);
    if (corr != 1.f) {
#pragma unroll
      for (int t = 0; t < 16; ++t) o[t][0] *= corr, o[t][1] *= corr, o[t][2] *= corr, o[t][3] *= corr;
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint32_t w0[4] = {vc[0][h].x, vc[0][h].y, vc[0][h].z, vc[0][h].w};
      const uint32_t w1[4] = {vc[1][h].x, vc[1][h].y, vc[1][h].z, vc[1][h].w};
      const uint32_t w2[4] = {vc[2][h].x, vc[2][h].y, vc[2][h].z, vc[2][h].w};
      const uint32_t w3[4] = {vc[3][h].x, vc[3][h].y, vc[3][h].z, vc[3][h].w};
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const uint32_t sel = (e & 1) ? 0x7632u : 0x5410u;
        const uint32_t b0 = __byte_perm(w0[e >> 1], w1[e >> 1], sel);
        const uint32_t b1 = __byte_perm(w2[e >> 1], w3[e >> 1], sel);
        mma_bf16_m16n8k16(o[8 * h + e], a0, a1, a2, a3, b0, b1);
      }
    }
    if (more) {
#pragma unroll
      for (int r = 0; r < 2; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) kc[r][c] = kn[r][c];
#pragma unroll
      for (int s = 0; s < 4; ++s) vc[s][0] = vn[s][0], vc[s][1] = vn[s][1];
    }
  }
  // Per-warp partial result. l is summed over the quad (m and corr were equal across it).
  l += __shfl_xor_sync(0xFFFFFFFFu, l, 1);
  l += __shfl_xor_sync(0xFFFFFFFFu, l, 2);
  if (gid < G) {
    if (tig == 0) part_ml[(warp * G + gid) * 2] = m, part_ml[(warp * G + gid) * 2 + 1] = l;
#pragma unroll
    for (int t = 0; t < 16; ++t) {
      const int h = t >> 3, e = t & 7;
      part_o[(warp * G + gid) * d + (2 * tig + 8 * h) * 8 + e] = o[t][0] + o[t][2];
      part_o[(warp * G + gid) * d + (2 * tig + 1 + 8 * h) * 8 + e] = o[t][1] + o[t][3];
    }
  }
  __syncthreads();
  if (S == 1) {
    attend_merge(part_ml, part_o, G, d, a.out + (size_t)unit * G * d);
    return;
  }
  attend_merge_cluster(part_ml, part_o, cta_ml, cta_o, G, d, S, rank, a.out + (size_t)unit * G * d);
}

// ------------------------------------------------------------------------------------------------ generic

__global__ void __launch_bounds__(kAttendThreads) attend_generic_kernel(const AttendArgs a) {
  extern __shared__ __align__(16) float asm_[];  // q as fp32 [G][d], then part_ml [warps][G][2], part_o [warps][G][d]
  const he_config& cfg = a.cfg;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int unit = blockIdx.y * cfg.n_kv_heads + blockIdx.x;
  const int d = cfg.head_dim, G = cfg.group_size, es = esize_of(cfg.dtype);
  const int fill = a.ca.fill[unit];
  float* qs = asm_;
  float* part_ml = qs + G * d;
  float* part_o = part_ml + kAttendWarps * G * 2;
  const int cpr = d * es / 16;
  for (int idx = tid; idx < G * cpr; idx += kAttendThreads)
    stage_chunk(qs + (idx / cpr) * d, static_cast<const char*>(a.q) + ((size_t)unit * G + idx / cpr) * d * es, idx % cpr, cfg.dtype);
  __syncthreads();
  const float scale = rsqrtf((float)d) * kLog2e;
  const char* Kb = static_cast<const char*>(a.ca.k_cache) + (size_t)unit * cfg.max_budget * d * es;
  const char* Vb = static_cast<const char*>(a.ca.v_cache) + (size_t)unit * cfg.max_budget * d * es;
  const int per = d / 32 + (d % 32 ? 1 : 0);  // channels per lane (<= 8): c = lane + 32 * i
  float m[kMaxGroup], l[kMaxGroup], o[kMaxGroup][kMaxDim / 32];
#pragma unroll
  for (int g = 0; g < kMaxGroup; ++g) {
    m[g] = -INFINITY;
    l[g] = 0.f;
#pragma unroll
    for (int i = 0; i < kMaxDim / 32; ++i) o[g][i] = 0.f;
  }
  auto elem = [&](const char* row, int c) -> float {
    return cfg.dtype == HE_DTYPE_BF16 ? bf16_bits_to_f32(reinterpret_cast<const uint16_t*>(row)[c])
                                      : reinterpret_cast<const float*>(row)[c];
  };
  for (int j = warp; j < fill; j += kAttendWarps) {
    const char* kr = Kb + (size_t)j * d * es;
    const char* vr = Vb + (size_t)j * d * es;
    float kv[kMaxDim / 32], vv[kMaxDim / 32];
#pragma unroll
    for (int i = 0; i < kMaxDim / 32; ++i) {
      const int c = lane + 32 * i;
      kv[i] = (i < per && c < d) ? elem(kr, c) : 0.f;
      vv[i] = (i < per && c < d) ? elem(vr, c) : 0.f;
    }
#pragma unroll
    for (int g = 0; g < kMaxGroup; ++g) {
      if (g < G) {
        float dot = 0.f;
#pragma unroll
        for (int i = 0; i < kMaxDim / 32; ++i) {
          const int c = lane + 32 * i;
          if (i < per && c < d) dot = fmaf(qs[g * d + c], kv[i], dot);
        }
        for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xFFFFFFFFu, dot, off);
        const float sc = dot * scale;
        const float mn = fmaxf(m[g], sc);
        const float corr = exp2f(m[g] - mn), p = exp2f(sc - mn);  // exp2f(-inf) = 0 on the first slot
        l[g] = l[g] * corr + p;
#pragma unroll
        for (int i = 0; i < kMaxDim / 32; ++i) o[g][i] = o[g][i] * corr + p * vv[i];
        m[g] = mn;
      }
    }
  }
#pragma unroll
  for (int g = 0; g < kMaxGroup; ++g) {
    if (g < G) {
      if (lane == 0) {
        part_ml[(warp * G + g) * 2] = m[g];
        part_ml[(warp * G + g) * 2 + 1] = l[g];
      }
#pragma unroll
      for (int i = 0; i < kMaxDim / 32; ++i) {
        const int c = lane + 32 * i;
        if (i < per && c < d) part_o[(warp * G + g) * d + c] = o[g][i];
      }
    }
  }
  __syncthreads();
  attend_merge(part_ml, part_o, G, d, a.out + (size_t)unit * G * d);
}

// ------------------------------------------------------------------------------------------------ attention loss
//
// he_attention_loss (Section 4.6 / Appendix B): 1 - the attention mass of the cached tokens, for each query head, under
// softmax(q . k_p / sqrt(d)) over ALL n = next_pos tokens seen so far. The dropped mass is summed directly (a token
// is dropped when no valid slot holds its position: a bitmap in shared memory), so a small loss is not the
// difference of two numbers close to one. One CTA per unit, a warp per token, online maximum as in he_attend.
struct LossArgs {
  he_config cfg;
  he_cache ca;
  const void* q;       // [B, Hkv*G, d]
  const void* k_full;  // strided [B, Hkv, n, d]
  long long s0, s1, s2;
  float* out;          // [B, Hkv*G]
};

__global__ void __launch_bounds__(kAttendThreads) attention_loss_kernel(const LossArgs a) {
  extern __shared__ __align__(16) float lsm_[];  // q as fp32 [G][d], partials [warps][G][3], bitmap of cached positions
  const he_config& cfg = a.cfg;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long unit = (long long)blockIdx.y * cfg.n_kv_heads + blockIdx.x;
  const int d = cfg.head_dim, G = cfg.group_size, es = esize_of(cfg.dtype);
  const int n = a.ca.next_pos[unit], fill = a.ca.fill[unit];
  float* qs = lsm_;
  float* part = qs + G * d;
  uint32_t* kept = reinterpret_cast<uint32_t*>(part + kAttendWarps * G * 3);
  const int cpr = d * es / 16;
  for (int idx = tid; idx < G * cpr; idx += kAttendThreads)
    stage_chunk(qs + (idx / cpr) * d, static_cast<const char*>(a.q) + (unit * G + idx / cpr) * d * es, idx % cpr, cfg.dtype);
  for (int i = tid; i < (n + 31) / 32; i += kAttendThreads) kept[i] = 0u;
  __syncthreads();
  for (int j = tid; j < fill; j += kAttendThreads) {
    const int p = a.ca.pos[unit * cfg.max_budget + j];
    if (p >= 0 && p < n) atomicOr(&kept[p >> 5], 1u << (p & 31));
  }
  __syncthreads();
  const float scale = rsqrtf((float)d) * kLog2e;
  const char* Kb = static_cast<const char*>(a.k_full) + ((long long)blockIdx.y * a.s0 + (long long)blockIdx.x * a.s1) * es;
  float m[kMaxGroup], lall[kMaxGroup], ldrop[kMaxGroup];
#pragma unroll
  for (int g = 0; g < kMaxGroup; ++g) m[g] = -INFINITY, lall[g] = 0.f, ldrop[g] = 0.f;
  const int per = (d + 31) / 32;
  for (int p = warp; p < n; p += kAttendWarps) {
    const char* kr = Kb + (long long)p * a.s2 * es;
    float kv[kMaxDim / 32];
#pragma unroll
    for (int i = 0; i < kMaxDim / 32; ++i) {
      const int c = lane + 32 * i;
      kv[i] = (i < per && c < d) ? (cfg.dtype == HE_DTYPE_BF16 ? bf16_bits_to_f32(reinterpret_cast<const uint16_t*>(kr)[c])
                                                                : reinterpret_cast<const float*>(kr)[c])
                                 : 0.f;
    }
    const bool dropped = ((kept[p >> 5] >> (p & 31)) & 1u) == 0u;
#pragma unroll
    for (int g = 0; g < kMaxGroup; ++g) {
      if (g < G) {
        float dot = 0.f;
#pragma unroll
        for (int i = 0; i < kMaxDim / 32; ++i) {
          const int c = lane + 32 * i;
          if (i < per && c < d) dot = fmaf(qs[g * d + c], kv[i], dot);
        }
        for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xFFFFFFFFu, dot, off);
        const float sc = dot * scale;
        const float mn = fmaxf(m[g], sc);
        const float corr = exp2f(m[g] - mn), w = exp2f(sc - mn);
        lall[g] = lall[g] * corr + w;
        ldrop[g] = ldrop[g] * corr + (dropped ? w : 0.f);
        m[g] = mn;
      }
    }
  }
  if (lane == 0) {
#pragma unroll
    for (int g = 0; g < kMaxGroup; ++g)
      if (g < G) {
        part[(warp * G + g) * 3] = m[g];
        part[(warp * G + g) * 3 + 1] = lall[g];
        part[(warp * G + g) * 3 + 2] = ldrop[g];
      }
  }
  __syncthreads();
  if (tid < G) {
    float M = -INFINITY;
    for (int w = 0; w < kAttendWarps; ++w) M = fmaxf(M, part[(w * G + tid) * 3]);
    float A = 0.f, D = 0.f;
    for (int w = 0; w < kAttendWarps; ++w) {
      const float mw = part[(w * G + tid) * 3];
      const float f = mw == -INFINITY ? 0.f : exp2f(mw - M);
      A += part[(w * G + tid) * 3 + 1] * f;
      D += part[(w * G + tid) * 3 + 2] * f;
    }
    a.out[unit * G + tid] = A > 0.f ? D / A : 0.f;
  }
}

// The same for bf16 keys with d = 128 and G <= 8: scores of 16 tokens at a time as warp-level MMAs fed straight from
// 16-byte global loads (the fragment scheme of attend_bf16_kernel), next group's rows requested before the current
// group's arithmetic. Dynamic shared memory: partials [warps][G][3] floats, then the bitmap of cached positions.
__global__ void __launch_bounds__(kAttendThreads) attention_loss_bf16_kernel(const LossArgs a) {
  extern __shared__ __align__(16) float lsm_[];
  constexpr int d = 128;
  const he_config& cfg = a.cfg;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, gid = lane >> 2, tig = lane & 3;
  const long long unit = (long long)blockIdx.y * cfg.n_kv_heads + blockIdx.x;
  const int G = cfg.group_size;
  const int n = a.ca.next_pos[unit], fill = a.ca.fill[unit];
  float* part = lsm_;
  uint32_t* kept = reinterpret_cast<uint32_t*>(part + kAttendWarps * G * 3);
  for (int i = tid; i < (n + 31) / 32; i += kAttendThreads) kept[i] = 0u;
  __syncthreads();
  for (int j = tid; j < fill; j += kAttendThreads) {
    const int p = a.ca.pos[unit * cfg.max_budget + j];
    if (p >= 0 && p < n) atomicOr(&kept[p >> 5], 1u << (p & 31));
  }
  __syncthreads();
  uint32_t qf[8][2];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    uint4 t = make_uint4(0u, 0u, 0u, 0u);
    if (gid < G) t = static_cast<const uint4*>(a.q)[(unit * G + gid) * (d / 8) + tig + 4 * c];
    qf[2 * c][0] = t.x, qf[2 * c][1] = t.y, qf[2 * c + 1][0] = t.z, qf[2 * c + 1][1] = t.w;
  }
  const float scale = rsqrtf((float)d) * kLog2e;
  const char* Kb = static_cast<const char*>(a.k_full) + ((long long)blockIdx.y * a.s0 + (long long)blockIdx.x * a.s1) * 2;
  const int last = n - 1;
  auto load_k = [&](int g0, uint4 (&kb)[2][4]) {  // rows past the end repeat the last row and are weighted by zero
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const uint4* row = reinterpret_cast<const uint4*>(Kb + (long long)min(g0 + gid + 8 * r, last) * a.s2 * 2);
#pragma unroll
      for (int c = 0; c < 4; ++c) kb[r][c] = ldg_stream16(row + tig + 4 * c);
    }
  };
  float m = -INFINITY, lall = 0.f, ldrop = 0.f;
  uint4 kc[2][4], kn[2][4];
  const int stride = 16 * kAttendWarps;
  int g0 = 16 * warp;
  if (g0 < n) load_k(g0, kc);
  for (; g0 < n; g0 += stride) {
    const bool more = g0 + stride < n;
    if (more) load_k(g0 + stride, kn);
    float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      mma_bf16_m16n8k16(s0, qf[2 * c][0], 0u, qf[2 * c][1], 0u, kc[0][c].x, kc[0][c].y);
      mma_bf16_m16n8k16(s1, qf[2 * c][0], 0u, qf[2 * c][1], 0u, kc[1][c].x, kc[1][c].y);
      mma_bf16_m16n8k16(s0, qf[2 * c + 1][0], 0u, qf[2 * c + 1][1], 0u, kc[0][c].z, kc[0][c].w);
      mma_bf16_m16n8k16(s1, qf[2 * c + 1][0], 0u, qf[2 * c + 1][1], 0u, kc[1][c].z, kc[1][c].w);
    }
    // this lane: head gid, tokens g0 + 2tig, + 1, + 8, + 9
    const int j = g0 + 2 * tig;
    const int tok[4] = {j, j + 1, j + 8, j + 9};
    const float sc[4] = {s0[0], s0[1], s1[0], s1[1]};
    float x[4];
    bool dropped[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      x[e] = tok[e] < n ? sc[e] * scale : -INFINITY;
      dropped[e] = tok[e] < n && ((kept[tok[e] >> 5] >> (tok[e] & 31)) & 1u) == 0u;
    }
    float gm = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
    gm = fmaxf(gm, __shfl_xor_sync(0xFFFFFFFFu, gm, 1));
    gm = fmaxf(gm, __shfl_xor_sync(0xFFFFFFFFu, gm, 2));  // finite: token g0 exists
    const float mn = fmaxf(m, gm);
    const float corr = exp2f(m - mn);
    float wa = 0.f, wd = 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float w = exp2f(x[e] - mn);
      wa += w;
      wd += dropped[e] ? w : 0.f;
    }
    lall = lall * corr + wa;
    ldrop = ldrop * corr + wd;
    m = mn;
    if (more) {
#pragma unroll
      for (int r = 0; r < 2; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) kc[r][c] = kn[r][c];
    }
  }
  lall += __shfl_xor_sync(0xFFFFFFFFu, lall, 1);
  lall += __shfl_xor_sync(0xFFFFFFFFu, lall, 2);
  ldrop += __shfl_xor_sync(0xFFFFFFFFu, ldrop, 1);
  ldrop += __shfl_xor_sync(0xFFFFFFFFu, ldrop, 2);
  if (gid < G && tig == 0) {
    part[(warp * G + gid) * 3] = m;
    part[(warp * G + gid) * 3 + 1] = lall;
    part[(warp * G + gid) * 3 + 2] = ldrop;
  }
  __syncthreads();
  if (tid < G) {
    float M = -INFINITY;
    for (int w = 0; w < kAttendWarps; ++w) M = fmaxf(M, part[(w * G + tid) * 3]);
    float A = 0.f, D = 0.f;
    for (int w = 0; w < kAttendWarps; ++w) {
      const float mw = part[(w * G + tid) * 3];
      const float f = mw == -INFINITY ? 0.f : exp2f(mw - M);
      A += part[(w * G + tid) * 3 + 1] * f;
      D += part[(w * G + tid) * 3 + 2] * f;
    }
    a.out[unit * G + tid] = A > 0.f ? D / A : 0.f;
  }
}

}  // namespace he
