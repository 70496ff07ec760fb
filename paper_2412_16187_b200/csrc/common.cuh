// Shared device helpers of the HashEvict kernels: constants, the projection order, and the Hamming-distance
// arithmetic of Eq. 5 (plain XOR+popcount, and a bit-plane form for groups of four query heads).
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "hashevict.h"

namespace he {

constexpr int kChunk = 32;       // channels per partial sum of the projection
constexpr int kMaxDim = 256;     // largest head_dim
constexpr int kMaxGroup = 8;     // largest group size
constexpr int kKeyIdxBits = 20;  // arg-max key = (distance part + 1) << 20 | (0xFFFFF - slot)
constexpr uint32_t kKeyIdxMask = (1u << kKeyIdxBits) - 1u;

__host__ __device__ inline int words_of(int b) { return (b + 31) >> 5; }
__host__ __device__ inline int esize_of(int dtype) { return dtype == HE_DTYPE_BF16 ? 2 : 4; }

// Bytes per slot of he_cache.codes in the packed layout (HE_FLAG_PACKED_CODES); 0 in the word layout, also where the
// two layouts are the same bytes (25..32 and 57..64 bits).
__host__ __device__ inline int packed_code_bytes(const he_config& cfg) {
  const int cb = (cfg.flags & HE_FLAG_PACKED_CODES) ? (cfg.hash_bits + 7) >> 3 : 0;
  return cb == 4 * words_of(cfg.hash_bits) ? 0 : cb;
}

// The code of one cache slot goes to he_cache.codes in the layout the config asks for. `code` holds WORDS words
// (constant indices only, so it may live in registers).
template <int WORDS>
__device__ __forceinline__ void store_slot_code(const he_config& cfg, uint32_t* codes, long long slot_idx,
                                                const uint32_t (&code)[WORDS]) {
  const int cb = packed_code_bytes(cfg);
  if (cb == 0) {
#pragma unroll
    for (int w = 0; w < WORDS; ++w) codes[slot_idx * WORDS + w] = code[w];
  } else {
    uint8_t* dst = reinterpret_cast<uint8_t*>(codes) + slot_idx * cb;
#pragma unroll
    for (int i = 0; i < 4 * WORDS; ++i)
      if (i < cb) dst[i] = (uint8_t)(code[i >> 2] >> (8 * (i & 3)));
  }
}

// Device-side trouble counter behind he_device_error_count: CTAs that gave up on a bounded wait and, in a build with
// -DHE_BOUNDS_CHECK, indices found out of range (stays 0 in a healthy run).
__device__ int g_tc_error = 0;

// Bounds checks of the debug build (build_cuda(debug=True) -> libhashevict_debug.so). Every slot or token index that a
// kernel computes or reads from memory before using it as an address goes through HE_IN_RANGE(i, n): true when
// 0 <= i < n. In the debug build a failed check is counted and the caller skips the access, so the kernel finishes
// and the host reads the count; the release build compiles the test away.
#ifdef HE_BOUNDS_CHECK
__device__ __forceinline__ bool he_in_range(long long i, long long n) {
  if (i >= 0 && i < n) return true;
  atomicAdd(&g_tc_error, 1);
  return false;
}
#define HE_IN_RANGE(i, n) ::he::he_in_range((long long)(i), (long long)(n))
#else
#define HE_IN_RANGE(i, n) true
#endif

// Device-side inputs the host cannot see are clamped where they are read: a prompt length into [0, Nmax] (the
// prompt-code scratch holds Nmax rows per unit), a budget into [0, Cmax]. A budget below 1 leaves nothing to store:
// the prefill calls then treat the sequence as empty and the decode calls leave its units untouched.
__device__ __forceinline__ int clamp_budget(int c, int cmax) { return min(max(c, 0), cmax); }
__device__ __forceinline__ int clamp_len(int n, int nmax, int c) { return c < 1 ? 0 : min(max(n, 0), nmax); }

__device__ __forceinline__ float bf16_bits_to_f32(uint32_t h) { return __uint_as_float(h << 16); }

__device__ __forceinline__ uint32_t word_mask(int b, int w) {
  const int n = b - 32 * w;
  return n >= 32 ? 0xFFFFFFFFu : (n <= 0 ? 0u : ((1u << n) - 1u));
}

// Writes 16 bytes of a row (8 bf16 or 4 fp32, already in registers) to fp32 shared memory.
__device__ __forceinline__ void store_chunk(float* dst, const uint4 raw, int chunk, int dtype) {
  if (dtype == HE_DTYPE_BF16) {
    float4* o = reinterpret_cast<float4*>(dst + chunk * 8);
    o[0] = make_float4(bf16_bits_to_f32(raw.x & 0xFFFFu), bf16_bits_to_f32(raw.x >> 16), bf16_bits_to_f32(raw.y & 0xFFFFu),
                       bf16_bits_to_f32(raw.y >> 16));
    o[1] = make_float4(bf16_bits_to_f32(raw.z & 0xFFFFu), bf16_bits_to_f32(raw.z >> 16), bf16_bits_to_f32(raw.w & 0xFFFFu),
                       bf16_bits_to_f32(raw.w >> 16));
  } else {
    *reinterpret_cast<float4*>(dst + chunk * 4) =
        make_float4(__uint_as_float(raw.x), __uint_as_float(raw.y), __uint_as_float(raw.z), __uint_as_float(raw.w));
  }
}

// Copies 16 bytes (8 bf16 or 4 fp32) of a row into fp32 shared memory.
__device__ __forceinline__ void stage_chunk(float* dst, const void* src_row, int chunk, int dtype) {
  store_chunk(dst, __ldg(reinterpret_cast<const uint4*>(src_row) + chunk), chunk, dtype);
}

// One LOP3 with an explicit truth table (a = 0xF0, b = 0xCC, c = 0xAA).
template <int LUT>
__device__ __forceinline__ uint32_t lop3(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, %4;" : "=r"(d) : "r"(a), "r"(b), "r"(c), "n"(LUT));
  return d;
}
// a ? b : c per bit
__device__ __forceinline__ uint32_t bitselect(uint32_t a, uint32_t b, uint32_t c) { return lop3<0xCA>(a, b, c); }

// ---------------------------------------------------------------------------------------------------------------
// Eq. 5 for a group of four query heads without four XOR+popcount passes.
//
// For one bit position let c in 0..4 be how many of the four query codes have a 1 there. A key bit h mismatches
// m = c of the queries when h = 0 and m = 4 - c when h = 1; the summed distance is D = sum over positions of m.
// Write m in binary. Its lowest bit is c mod 2 whatever h is, so that plane contributes the same amount to every
// slot: a per-step constant. Only the 2s plane and the 4s plane depend on the key:
//     m1 = h ? [c in {1,2}] : [c in {2,3}]        m2 = h ? [c == 0] : [c == 4]
// so  D = popc(c0) + 2 * popc(select(h, A1, B1)) + 4 * popc(select(h, A2, B2)),
// two selects and two popcounts per code word instead of four XORs and four popcounts. Exact integer identity.
// ---------------------------------------------------------------------------------------------------------------
struct Planes4 {
  uint32_t a1, a2, b1, b2;  // per code word: planes used when the key bit is 1 (a*) or 0 (b*)
};

__device__ __forceinline__ Planes4 make_planes4(uint32_t q0, uint32_t q1, uint32_t q2, uint32_t q3, uint32_t* parity) {
  const uint32_t s01 = q0 ^ q1, a01 = q0 & q1, s23 = q2 ^ q3, a23 = q2 & q3;
  const uint32_t c0 = s01 ^ s23, k = s01 & s23;
  const uint32_t c1 = a01 ^ a23 ^ k;  // count in {2, 3}
  const uint32_t c2 = a01 & a23;      // count == 4
  Planes4 p;
  p.b1 = c1;
  p.b2 = c2;
  p.a1 = c0 ^ c1;               // count in {1, 2}
  p.a2 = ~(q0 | q1 | q2 | q3);  // count == 0 (positions beyond b have key bit 0, so they never select this plane)
  *parity = c0;
  return p;
}

// Key-dependent half of the group-of-four distance: (D - popc(parity planes)) / 2.
template <int WORDS>
__device__ __forceinline__ int half_distance4(const uint32_t (&h)[WORDS], const Planes4 (&p)[WORDS]) {
  if (WORDS == 2) {
    // two code words: add the planes of equal weight with carry-save logic first, so three popcounts suffice
    const uint32_t p1a = bitselect(h[0], p[0].a1, p[0].b1), p1b = bitselect(h[WORDS - 1], p[WORDS - 1].a1, p[WORDS - 1].b1);
    const uint32_t p2a = bitselect(h[0], p[0].a2, p[0].b2), p2b = bitselect(h[WORDS - 1], p[WORDS - 1].a2, p[WORDS - 1].b2);
    const uint32_t s1 = p1a ^ p1b, c1 = p1a & p1b;  // weight 1, carry of weight 2
    const uint32_t s2 = lop3<0x96>(c1, p2a, p2b);     // weight 2: three-way xor
    const uint32_t c2 = lop3<0xE8>(c1, p2a, p2b);     // weight 4: majority
    return __popc(s1) + 2 * __popc(s2) + 4 * __popc(c2);
  }
  int d = 0;
#pragma unroll
  for (int w = 0; w < WORDS; ++w)
    d += __popc(bitselect(h[w], p[w].a1, p[w].b1)) + 2 * __popc(bitselect(h[w], p[w].a2, p[w].b2));
  return d;
}

// Plain form for any group size: D = sum_g popc(h ^ q_g). `q` points at G * WORDS words (shared memory or registers).
template <int WORDS>
__device__ __forceinline__ int plain_distance(const uint32_t (&h)[WORDS], const uint32_t* q, int G) {
  int d = 0;
  for (int g = 0; g < G; ++g)
#pragma unroll
    for (int w = 0; w < WORDS; ++w) d += __popc(h[w] ^ q[g * WORDS + w]);
  return d;
}

}  // namespace he

namespace he {

// Per-step query context: built once from the step's query codes, then asked for the distance of each slot.
// rank(h) is monotone in the distance D and cheap; dist(rank) returns the exact D of Eq. 5.
// A context can be stored as kRecWords words (build) and loaded back (load), so that one warp can prepare the
// contexts of many prompt tokens ahead of the scan.
template <int WORDS, int GT>
struct QueryCtx;

template <int WORDS>
struct QueryCtx<WORDS, 4> {
  static constexpr int kRecWords = 4 * WORDS + 1;
  Planes4 p[WORDS];
  int base;
  __device__ __forceinline__ static void build(uint32_t* rec, const uint32_t* q, int) {
    int base = 0;
#pragma unroll
    for (int w = 0; w < WORDS; ++w) {
      uint32_t parity;
      const Planes4 pl = make_planes4(q[w], q[WORDS + w], q[2 * WORDS + w], q[3 * WORDS + w], &parity);
      rec[4 * w] = pl.a1;
      rec[4 * w + 1] = pl.a2;
      rec[4 * w + 2] = pl.b1;
      rec[4 * w + 3] = pl.b2;
      base += __popc(parity);
    }
    rec[4 * WORDS] = (uint32_t)base;
  }
  __device__ __forceinline__ void load(const uint32_t* rec, int) {
#pragma unroll
    for (int w = 0; w < WORDS; ++w) {
      p[w].a1 = rec[4 * w];
      p[w].a2 = rec[4 * w + 1];
      p[w].b1 = rec[4 * w + 2];
      p[w].b2 = rec[4 * w + 3];
    }
    base = (int)rec[4 * WORDS];
  }
  __device__ __forceinline__ int rank(const uint32_t (&h)[WORDS]) const { return half_distance4<WORDS>(h, p); }
  __device__ __forceinline__ int dist(int rank) const { return base + 2 * rank; }
};

template <int WORDS>
struct QueryCtx<WORDS, 1> {
  static constexpr int kRecWords = WORDS;
  uint32_t q[WORDS];
  __device__ __forceinline__ static void build(uint32_t* rec, const uint32_t* q, int) {
#pragma unroll
    for (int w = 0; w < WORDS; ++w) rec[w] = q[w];
  }
  __device__ __forceinline__ void load(const uint32_t* rec, int) {
#pragma unroll
    for (int w = 0; w < WORDS; ++w) q[w] = rec[w];
  }
  __device__ __forceinline__ int rank(const uint32_t (&h)[WORDS]) const {
    int d = 0;
#pragma unroll
    for (int w = 0; w < WORDS; ++w) d += __popc(h[w] ^ q[w]);
    return d;
  }
  __device__ __forceinline__ int dist(int rank) const { return rank; }
};

template <int WORDS>
struct QueryCtx<WORDS, 0> {
  static constexpr int kRecWords = kMaxGroup * WORDS;
  const uint32_t* q;
  int G;
  __device__ __forceinline__ static void build(uint32_t* rec, const uint32_t* q, int G) {
#pragma unroll
    for (int i = 0; i < kMaxGroup * WORDS; ++i)
      if (i < G * WORDS) rec[i] = q[i];
  }
  __device__ __forceinline__ void load(const uint32_t* rec, int G_) {
    q = rec;  // stays in shared memory
    G = G_;
  }
  __device__ __forceinline__ int rank(const uint32_t (&h)[WORDS]) const { return plain_distance<WORDS>(h, q, G); }
  __device__ __forceinline__ int dist(int rank) const { return rank; }
};

// block-wide arg-max of packed keys: redux.sync inside each warp, one barrier, redux.sync over the warp results
__device__ __forceinline__ uint32_t block_max_key(uint32_t key, uint32_t* wbuf, int lane, int warp, int nwarps) {
  key = __reduce_max_sync(0xFFFFFFFFu, key);
  if (lane == 0) wbuf[warp] = key;
  __syncthreads();
  return __reduce_max_sync(0xFFFFFFFFu, lane < nwarps ? wbuf[lane] : 0u);
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
// Waits until at most `pending` of this thread's commit groups are still in flight (pending must fold to a constant).
__device__ __forceinline__ void cp_async_wait_pending(int pending) {
  switch (pending) {
    case 0: asm volatile("cp.async.wait_group 0;\n" ::: "memory"); break;
    case 1: asm volatile("cp.async.wait_group 1;\n" ::: "memory"); break;
    case 2: asm volatile("cp.async.wait_group 2;\n" ::: "memory"); break;
    case 3: asm volatile("cp.async.wait_group 3;\n" ::: "memory"); break;
    case 4: asm volatile("cp.async.wait_group 4;\n" ::: "memory"); break;
    case 5: asm volatile("cp.async.wait_group 5;\n" ::: "memory"); break;
    case 6: asm volatile("cp.async.wait_group 6;\n" ::: "memory"); break;
    default: asm volatile("cp.async.wait_group 7;\n" ::: "memory"); break;
  }
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;\n" ::: "memory"); }

// Asks for `bytes` (a multiple of 16, from a 16-byte aligned address) to be brought into L2. A hint: no data returns.
__device__ __forceinline__ void l2_prefetch_bulk(const void* gmem, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;\n" ::"l"(gmem), "r"(bytes) : "memory");
}

// Programmatic dependent launch: a kernel launched with the programmatic-serialization attribute may start while
// the previous kernel of the stream is still draining. Everything that touches memory another kernel may have
// written comes after griddep_wait(); only W (read-only while a cache is in use) is read before it.
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

}  // namespace he
