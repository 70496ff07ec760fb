// Eq. 2 on many bf16 rows with the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor memory).
//
// Why tensor cores here and nowhere else on this path: the projection X[rows, d] * W[d, b] is the one dense
// contraction, and at b >= 16 its arithmetic intensity (b flop per input byte) puts the CUDA-core kernel on the
// fp32 FMA pipe instead of on HBM (profiles/: DRAM at ~5 % of peak). Exactness is kept by splitting the fp32 W
// into three bf16 terms W = W1 + W2 + W3 (each residual is exact in fp32, so the three terms carry all 24
// significand bits): x is bf16, every product x * W_t is exact, and only the fp32 accumulation rounds. The sign
// of the result may therefore differ from exact arithmetic only within the same 1e-5 * |x| * |w| band that the
// fp32 CUDA-core kernel is allowed; the parity tests check every hashed bit against that rule.
//
// One persistent CTA per SM, 192 threads, warp-specialised:
//   warps 0-3  epilogue: tcgen05.ld the 128 x N fp32 accumulator (one row per thread), sign bits -> code words
//   warp 4     producer: one thread issues a TMA tensor copy per 64-channel half of a 128-row tile (the hardware
//              applies the 128-byte swizzle and signals the stage's mbarrier with the byte count); when no tensor
//              map can be built for the caller's strides the warp falls back to 16-byte cp.async copies
//   warp 5     one thread issues 3 terms x d/16 tcgen05.mma (M = 128, N = 32|64, K = 16) per tile and commits
// Four shared-memory stages for X, W's three terms resident in shared memory, two accumulators in tensor memory
// so the epilogue of tile i overlaps the MMAs of tile i+1. Every wait on an mbarrier is bounded: when a limit is
// hit the CTA raises a flag, all roles leave their loops, tensor memory is released and the kernel returns.
#pragma once
#include <cuda.h>  // CUtensorMap (types only; the encoder is fetched through the runtime)

#include "common.cuh"
#include "hash_kernels.cuh"

namespace he {

constexpr int kTcThreads = 192;
constexpr int kTcRows = 128;          // rows per tile = MMA M
constexpr int kTcStages = 4;          // X tiles in flight
constexpr int kTcLag = 2;             // cp.async groups the producer leaves in flight before publishing a stage
constexpr uint32_t kTcSpinLimit = 1u << 22;
constexpr int kTcLenCache = 2048;     // sequences whose prompt length and budget are cached in shared memory


__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait. Returns false (and raises the CTA-wide abort flag) when the limit is hit or another role aborted.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < kTcSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

// Bounded wait that neither reads nor raises the abort flag: used on the way out of an aborted CTA, to let work that
// is already in flight finish before shared or tensor memory is given up. Gives up silently after the same limit.
__device__ __forceinline__ void mbar_drain(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kTcSpinLimit; ++i)
    if (mbar_try_wait(bar, parity)) return;
}

// Bounded wait on two barriers at once: both are polled in the same loop, so their latencies overlap (one polling
// round trip costs a couple of hundred cycles even when the phase has long completed).
__device__ __forceinline__ bool mbar_wait2(uint32_t bar_a, uint32_t parity_a, uint32_t bar_b, uint32_t parity_b,
                                           volatile int* abort_flag) {
  bool ok_a = false, ok_b = false;
  for (uint32_t i = 0; i < kTcSpinLimit; ++i) {
    if (!ok_a) ok_a = mbar_try_wait(bar_a, parity_a);
    if (!ok_b) ok_b = mbar_try_wait(bar_b, parity_b);
    if (ok_a && ok_b) return true;
    if (*abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// TMA tile copy global -> shared for this CTA alone, completion counted in bytes on `bar`
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tmap, int c0, int c1, int c2, int c3, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"((uint32_t)accumulate)
      : "memory");
}
// 32 consecutive fp32 columns of this thread's tensor-memory lane
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_k128(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) /* leading offset (unused with swizzle) */ |
         ((uint64_t)(1024 >> 4) << 32) /* stride between 8-row groups */ | (1ull << 46) /* descriptor version */ |
         (2ull << 61) /* SWIZZLE_128B */;
}

__device__ __forceinline__ uint16_t bf16_rne_bits(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u & 0x7F800000u) == 0x7F800000u) return (uint16_t)(u >> 16);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

// One element of W -> its three bf16 terms at their places in the image: per 64-channel half one K-major operand of
// 3N rows (term 1's N bit rows, then term 2's, then term 3's), 128 bytes per row with the 128-byte swizzle. The three
// terms are thus three column groups of ONE MMA (N = 96 or 192): a third of the instructions, and the kernel is bound
// by MMA issue.
__device__ __forceinline__ void w_image_element(const float* W, int d, int b, int N, int idx, unsigned char* image) {
  const int c = idx / N, i = idx % N, tile_bytes = N * 128;
  const float w = i < b ? __ldg(W + (long long)c * b + i) : 0.f;
  const uint16_t w1 = bf16_rne_bits(w);
  const float r1 = w - bf16_bits_to_f32(w1);
  const uint16_t w2 = bf16_rne_bits(r1);
  const float r2 = r1 - bf16_bits_to_f32(w2);
  const uint16_t w3 = bf16_rne_bits(r2);
  const int kh = c / 64, kk = c % 64;
  const int off = (i / 8) * 1024 + (i % 8) * 128 + (((kk / 8) ^ (i % 8)) * 16) + (kk % 8) * 2;
  *reinterpret_cast<uint16_t*>(image + (kh * 3 + 0) * tile_bytes + off) = w1;
  *reinterpret_cast<uint16_t*>(image + (kh * 3 + 1) * tile_bytes + off) = w2;
  *reinterpret_cast<uint16_t*>(image + (kh * 3 + 2) * tile_bytes + off) = w3;
}

// The image in global memory, built once per call when the caller has scratch for it (kWImageBytes at most).
constexpr size_t kWImageBytes = 3 * 2 * 64 * 128;  // three terms, d = 128, N = 64
__global__ void build_w_image_kernel(const float* W, int d, int b, int N, unsigned char* image) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < d * N) w_image_element(W, d, b, N, idx, image);
}

// Which rows a tile covers and where its codes go (same segment rules as hash_rows_kernel).
struct TcTile {
  const char* base;
  long long stride;  // elements between rows
  long long row0;
  int nrows;
  long long out_base, out_stride;
  int c2, c3;  // tensor-map coordinates of the segment (head, sequence)
  int second;  // flat rows: the tile lies in the job's second range (its own tensor map)
};

// Dense schedule (prompt modes, batch within kTcLenCache): s_pref[s] counts the non-empty tiles of the sequences before
// s (all heads), so tile numbers below s_pref[nseq] name non-empty tiles only and a strided walk over them gives every
// CTA the same number of real tiles whatever the prompt lengths. `hint` is the caller's sequence cursor: tile numbers
// only grow, so the search is a short walk forward. With nseq_dense = 0 tiles are numbered (segment, tile in segment)
// and the empty ones are skipped.
template <int WORDS>
__device__ __forceinline__ bool tc_tile(const HashJob& job, long long t, long long tiles_per_seg, TcTile* o,
                                        const int* s_len, const int* s_bud, const unsigned* s_pref, int nseq_dense, int* hint) {
  // 64-bit division is emulated and every role calls this once per tile: keep it to 32 bits whenever the counts fit
  int seg, s_d = 0, hh_d = 0;  // dense schedule: sequence and head are known without dividing again
  long long ti;
  if (nseq_dense > 0) {
    int sq = *hint;
    const unsigned tt = (unsigned)t;
    while (sq + 1 < nseq_dense && s_pref[sq + 1] <= tt) ++sq;
    *hint = sq;
    const unsigned rem = tt - s_pref[sq];
    const unsigned nt = (s_pref[sq + 1] - s_pref[sq]) / (unsigned)job.heads;  // tiles per head of this sequence (> 0 here)
    const unsigned hh = rem / nt;
    seg = 0;
    s_d = sq;
    hh_d = (int)hh;
    ti = (long long)(rem - hh * nt);
  } else if (job.mode == 0) {
    seg = 0;
    ti = t;
  } else if (t < 0x7FFFFFFFll && tiles_per_seg < 0x7FFFFFFFll) {
    const unsigned tt = (unsigned)t, tp = (unsigned)tiles_per_seg;
    seg = (int)(tt / tp);
    ti = (long long)(tt - (unsigned)seg * tp);
  } else {
    seg = (int)(t / tiles_per_seg);
    ti = t % tiles_per_seg;
  }
  long long r_begin, r_end;
  o->second = 0;
  if (job.mode == 0) {
    const long long tiles1 = (job.rows + kTcRows - 1) / kTcRows;
    o->second = ti >= tiles1 ? 1 : 0;
    if (o->second) ti -= tiles1;
    o->base = static_cast<const char*>(o->second ? job.x2 : job.x);
    o->stride = job.row_stride;
    r_begin = 0;
    r_end = o->second ? job.rows2 : job.rows;
    o->out_base = o->second ? job.rows * WORDS : 0;
    o->out_stride = WORDS;
    o->c2 = 0;
    o->c3 = 0;
  } else {
    const int s = nseq_dense > 0 ? s_d : seg / job.heads, hh = nseq_dense > 0 ? hh_d : seg % job.heads;
    // lengths come from the CTA's shared-memory copy when the batch fits it: skipping an empty tile is then cheap
    const long long C = s < kTcLenCache ? s_bud[s] : max(job.budget[s], 0);
    const long long N = s < kTcLenCache ? s_len[s] : clamp_len(job.prompt_len[s], job.Nmax, (int)min(C, 1LL));
    o->c2 = hh;
    o->c3 = s;
    o->base = static_cast<const char*>(job.x) + (s * job.s0 + hh * job.s1) * 2;
    o->stride = job.s2;
    r_end = N;
    if (job.mode == 1) {
      r_begin = 0;
      o->out_base = ((long long)s * job.Hkv + hh) * job.Nmax * WORDS;
      o->out_stride = WORDS;
    } else {
      r_begin = job.q_all ? 0 : (C < N ? C : N);
      const long long unit = (long long)s * job.Hkv + hh / job.G;
      o->out_base = (unit * job.Nmax * job.G + hh % job.G) * WORDS;
      o->out_stride = (long long)job.G * WORDS;
    }
  }
  o->row0 = r_begin + ti * kTcRows;
  if (o->row0 >= r_end) return false;
  o->nrows = (int)((r_end - o->row0) < kTcRows ? (r_end - o->row0) : kTcRows);
  return true;
}

// Dynamic shared memory (after rounding the base up to 1024 bytes):
//   B: 3 terms x KH halves x [N rows x 128 bytes]      A: kTcStages x KH halves x [128 rows x 128 bytes]
template <int WORDS, bool TMA>
__global__ void __launch_bounds__(kTcThreads, 1) hash_rows_tc_kernel(const HashJob job, long long total_tiles,
                                                                     long long tiles_per_seg,
                                                                     const __grid_constant__ CUtensorMap tmap,
                                                                     const __grid_constant__ CUtensorMap tmap2) {
  constexpr int N = 32 * WORDS;
  constexpr int kAccCols = 3 * N;                          // one accumulator: the three terms side by side
  constexpr int kTmemCols = 2 * kAccCols <= 256 ? 256 : 512;  // two accumulators, rounded up to a power of two
  extern __shared__ unsigned char tc_smem_raw[];
  __shared__ __align__(8) unsigned long long bars[2 * kTcStages + 5];  // the last one: drain barrier of the abort path
  __shared__ uint32_t tmem_base_s;
  __shared__ volatile int abort_flag;
  __shared__ int s_len[kTcLenCache], s_bud[kTcLenCache];
  __shared__ unsigned s_pref[kTcLenCache + 1];  // dense schedule: non-empty tiles (all heads) of the sequences before s
  __shared__ int s_nseq_dense;

  // Programmatic dependent launch (used by the large-batch decode step): a kernel launched behind this one may
  // start right away; this kernel in turn finishes only after the kernel before it has (see the end).
  griddep_launch_dependents();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int d = job.d, b = job.b;
  const int KH = d / 64;  // 64-channel halves (128 bytes of bf16 each)
  // rounded up to 1024 bytes by an offset from the array itself: the accesses stay shared-memory accesses
  unsigned char* smem = tc_smem_raw + ((1024u - (smem_u32(tc_smem_raw) & 1023u)) & 1023u);
  unsigned char* Bs = smem;
  const int b_tile_bytes = N * 128;
  unsigned char* As = Bs + 3 * KH * b_tile_bytes;  // N * 128 is a multiple of 1024 for N = 32, 64
  const int a_half_bytes = kTcRows * 128;
  const int a_stage_bytes = KH * a_half_bytes;

  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kTcStages + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kTcStages + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kTcStages + 2 + a); };
  const uint32_t drain_bar = bar0 + 8u * (2 * kTcStages + 4);

  if (tid == 0) {
    abort_flag = 0;
    mbar_init(drain_bar, 1);
    for (int s = 0; s < kTcStages; ++s) {
      mbar_init(full_bar(s), TMA ? 1 : 32);  // TMA: one arrive + byte count; cp.async: every producer lane arrives
      mbar_init(empty_bar(s), 1);  // tcgen05.commit
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);   // tcgen05.commit
      mbar_init(tempty_bar(a), 4);  // one lane of each epilogue warp
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) {  // tensor memory: two accumulators of N columns each -> 2N columns (a power of two >= 32)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  const int nseq = job.mode != 0 ? (int)(total_tiles / tiles_per_seg) / job.heads : 0;
  if (job.mode != 0) {
    for (int i = threadIdx.x; i < nseq && i < kTcLenCache; i += kTcThreads) {
      s_bud[i] = max(job.budget[i], 0);
      s_len[i] = clamp_len(job.prompt_len[i], job.Nmax, min(s_bud[i], 1));
    }
  }
  if (tid == 0) s_nseq_dense = 0;
  // W -> three bf16 terms, transposed to [bit][channel] (K-major), 128B-swizzled; columns beyond b are zero.
  // Either copied from an image that a one-block-per-slice kernel prepared once for this call, or built here.
  if (job.w_image != nullptr) {
    const uint4* src = static_cast<const uint4*>(job.w_image);
    uint4* dst = reinterpret_cast<uint4*>(Bs);
    for (int i = tid; i < 3 * KH * b_tile_bytes / 16; i += kTcThreads) dst[i] = __ldg(src + i);
  } else {
    for (int idx = tid; idx < d * N; idx += kTcThreads) w_image_element(job.W, d, b, N, idx, Bs);
  }
  fence_proxy_async();  // the generic-proxy writes above are read by the tensor core through the async proxy
  if (job.mode != 0 && nseq <= kTcLenCache && total_tiles < 0x7FFFFFFFll) {
    __syncthreads();  // the cached lengths are complete
    if (warp == 0) {  // exclusive prefix over the sequences' tile counts, 32 at a time
      unsigned run = 0;
      for (int i0 = 0; i0 < nseq; i0 += 32) {
        const int i = i0 + lane;
        unsigned cnt = 0;
        if (i < nseq) {
          const long long Ni = s_len[i], Ci = s_bud[i];
          const long long r0 = (job.mode == 1 || job.q_all) ? 0 : (Ci < Ni ? Ci : Ni);
          long long nt = Ni > r0 ? (Ni - r0 + kTcRows - 1) / kTcRows : 0;
          if (nt > tiles_per_seg) nt = tiles_per_seg;
          cnt = (unsigned)nt * (unsigned)job.heads;
        }
        unsigned inc = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned v = __shfl_up_sync(0xFFFFFFFFu, inc, o);
          if (lane >= o) inc += v;
        }
        if (i < nseq) s_pref[i] = run + inc - cnt;
        run += __shfl_sync(0xFFFFFFFFu, inc, 31);
      }
      if (lane == 0) {
        s_pref[nseq] = run;
        s_nseq_dense = nseq;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  const int nseq_dense = s_nseq_dense;
  const long long n_sched = nseq_dense > 0 ? (long long)s_pref[nseq_dense] : total_tiles;  // tile numbers this grid walks
  int cursor = 0;  // this thread's sequence cursor of the dense schedule

  // Flat rows and the dense schedule number real tiles only, so every role walks t = blockIdx.x, + gridDim.x, ... and all
  // of them are tiles. There the producer warp and the epilogue warps work out the tiles' coordinates 32 at a time, a
  // lane per tile, and hand them round by shuffle: done by one thread per tile, that index arithmetic (a search, a
  // division, 64-bit products) was the longest dependent chain of the kernel's per-tile work.
  const bool batched = nseq_dense > 0 || job.mode == 0;
  if (warp == 4 && TMA) {
    // ------------------------------------------------------------------ producer (TMA, one thread issues)
    int it = 0;
    auto issue = [&](int row0, int c2, int c3, int second) -> bool {  // lane 0
      const int s = it % kTcStages;
      if (!mbar_wait(empty_bar(s), ((it / kTcStages) & 1) ^ 1, &abort_flag)) return false;
      mbar_arrive_expect_tx(full_bar(s), (uint32_t)a_stage_bytes);
      // rows past the tensor's extent are filled with zeros by the copy engine; their codes are not stored
      for (int kh = 0; kh < KH; ++kh)
        tma_load_4d(smem_u32(As + s * a_stage_bytes + kh * a_half_bytes), second ? &tmap2 : &tmap, kh * 64, row0, c2, c3, full_bar(s));
      return true;
    };
    if (batched) {
      bool alive = true;
      for (long long tb = blockIdx.x; tb < n_sched && alive; tb += 32LL * gridDim.x) {
        const long long t = tb + (long long)lane * gridDim.x;
        int row0 = 0, c2 = 0, c3 = 0, second = 0;
        TcTile tl;
        if (t < n_sched && tc_tile<WORDS>(job, t, tiles_per_seg, &tl, s_len, s_bud, s_pref, nseq_dense, &cursor))
          row0 = (int)tl.row0, c2 = tl.c2, c3 = tl.c3, second = tl.second;
        const long long left = (n_sched - tb + gridDim.x - 1) / gridDim.x;
        const int cnt = left < 32 ? (int)left : 32;
        for (int j = 0; j < cnt && alive; ++j) {
          const int r0 = __shfl_sync(0xFFFFFFFFu, row0, j), a2 = __shfl_sync(0xFFFFFFFFu, c2, j);
          const int a3 = __shfl_sync(0xFFFFFFFFu, c3, j), sc = __shfl_sync(0xFFFFFFFFu, second, j);
          int ok = 1;
          if (lane == 0) ok = issue(r0, a2, a3, sc) ? 1 : 0;
          alive = __shfl_sync(0xFFFFFFFFu, ok, 0) != 0;
          if (alive) ++it;
        }
      }
    } else if (lane == 0) {
      for (long long t = blockIdx.x; t < n_sched; t += gridDim.x) {
        TcTile tl;
        if (!tc_tile<WORDS>(job, t, tiles_per_seg, &tl, s_len, s_bud, s_pref, nseq_dense, &cursor)) continue;
        if (!issue((int)tl.row0, tl.c2, tl.c3, tl.second)) break;
        ++it;
      }
    }
    // A CTA that gives up must not hand its shared memory back while a tile copy into it is still under way: wait
    // (bounded) for the copies of the stages armed last.
    if (lane == 0 && abort_flag)
      for (int u = it > kTcStages ? it - kTcStages : 0; u < it; ++u) mbar_drain(full_bar(u % kTcStages), (u / kTcStages) & 1);
  } else if (warp == 4) {
    // ------------------------------------------------------------------ producer (cp.async fallback)
    int it = 0;                // tiles this CTA has started
    int published = 0;         // tiles whose stage has been handed to the MMA thread
    bool ok = true;
    auto publish = [&]() {
      fence_proxy_async();
      mbar_arrive(full_bar(published % kTcStages));
      ++published;
    };
    for (long long t = blockIdx.x; t < n_sched && ok; t += gridDim.x) {
      TcTile tl;
      if (!tc_tile<WORDS>(job, t, tiles_per_seg, &tl, s_len, s_bud, s_pref, nseq_dense, &cursor)) continue;
      const int s = it % kTcStages;
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(empty_bar(s), ((it / kTcStages) & 1) ^ 1, &abort_flag));  // warp-uniform
      if (!ok) break;
      unsigned char* a_stage = As + s * a_stage_bytes;
      const int cpr = d / 8;  // 16-byte chunks per row
      for (int idx = lane; idx < kTcRows * cpr; idx += 32) {
        const int r = idx / cpr, c = idx % cpr;
        const int rs = r < tl.nrows ? r : tl.nrows - 1;  // rows past the end repeat the last row; their codes are not stored
        const char* src = tl.base + ((tl.row0 + rs) * tl.stride) * 2 + c * 16;
        unsigned char* dst = a_stage + (c / 8) * a_half_bytes + (r / 8) * 1024 + (r % 8) * 128 + (((c % 8) ^ (r % 8)) * 16);
        cp_async16(dst, src);
      }
      cp_async_commit();
      ++it;
      if (it - published > kTcLag) {
        asm volatile("cp.async.wait_group %0;" ::"n"(kTcLag) : "memory");
        publish();
      }
    }
    cp_async_wait_all();
    while (published < it) publish();
  } else if (warp == 5) {
    // ------------------------------------------------------------------ MMA issue (one thread)
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) /* fp32 accumulate */ | (1u << 7) /* A bf16 */ | (1u << 10) /* B bf16 */ |
                             ((uint32_t)(kAccCols >> 3) << 17) | ((uint32_t)(kTcRows >> 4) << 24);
      const uint64_t b_desc0 = umma_desc_k128(smem_u32(Bs));
      int it = 0;
      for (long long t = blockIdx.x; t < n_sched; t += gridDim.x) {
        // flat rows and the dense schedule number real tiles only; otherwise empty tiles are skipped like the other
        // roles skip them (this thread needs nothing else of the tile, so it avoids the index arithmetic)
        if (job.mode != 0 && nseq_dense == 0) {
          TcTile tl;
          if (!tc_tile<WORDS>(job, t, tiles_per_seg, &tl, s_len, s_bud, s_pref, nseq_dense, &cursor)) continue;
        }
        const int s = it % kTcStages, acc = it & 1;
        // the epilogue has drained this accumulator and the stage's rows have landed
        if (!mbar_wait2(tempty_bar(acc), ((it >> 1) & 1) ^ 1, full_bar(s), (it / kTcStages) & 1, &abort_flag)) break;
        tc_fence_after();
        // Descriptors differ only in their 14-bit start-address field, so each MMA's pair is the tile's base
        // descriptor plus a small constant: the issuing thread spends a few instructions per MMA, not dozens.
        const uint64_t a_desc0 = umma_desc_k128(smem_u32(As + s * a_stage_bytes));
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kAccCols);
#pragma unroll
        for (int kh = 0; kh < 2; ++kh) {
          if (kh < KH) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)  // K = 16 bf16 = 32 bytes per instruction inside the 128-byte swizzle span
              tc_mma_bf16(d_tmem, a_desc0 + (uint64_t)((kh * (kTcRows * 128) + ks * 32) >> 4),
                          b_desc0 + (uint64_t)((kh * 3 * (N * 128) + ks * 32) >> 4), idesc, !(kh == 0 && ks == 0));
          }
        }
        tc_commit(empty_bar(s));    // the stage may be refilled once these MMAs have read it
        tc_commit(tfull_bar(acc));  // and the accumulator is complete
        ++it;
      }
      // ... nor free tensor memory under an MMA that is still writing it: one more commit tracks everything this thread
      // has issued, and its completion is awaited (bounded) before the CTA goes on to the deallocation.
      if (abort_flag) {
        tc_commit(drain_bar);
        mbar_drain(drain_bar, 0);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 0-3, one row per thread)
    int it = 0;
    // one tile: `obase` = index of its first row's first code word in job.out, `ostride` words between rows
    auto epi_tile = [&](long long obase, int ostride, int nrows) -> bool {
      const int acc = it & 1;
      if (!__all_sync(0xFFFFFFFFu, mbar_wait(tfull_bar(acc), (it >> 1) & 1, &abort_flag))) return false;  // warp-uniform
      tc_fence_after();
      uint32_t code[WORDS];
#pragma unroll
      for (int w = 0; w < WORDS; ++w) {
        uint32_t v1[32], v2[32], v3[32];
        const uint32_t base = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(acc * kAccCols + w * 32);
        tc_ld32(base, v1);
        tc_ld32(base + N, v2);
        tc_ld32(base + 2 * N, v3);
        tc_wait_ld();
        uint32_t word = 0u;
#pragma unroll
        for (int i = 0; i < 32; ++i) {  // the three terms' partial sums, smallest term first
          const float p = (__uint_as_float(v3[i]) + __uint_as_float(v2[i])) + __uint_as_float(v1[i]);
          word |= (p >= 0.f ? 1u : 0u) << i;
        }
        code[w] = word & word_mask(b, w);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
      const int r = warp * 32 + lane;
      if (r < nrows) {
        uint32_t* o = job.out + obase + (long long)r * ostride;
#pragma unroll
        for (int w = 0; w < WORDS; ++w) o[w] = code[w];
      }
      return true;
    };
    if (batched) {
      bool alive = true;
      for (long long tb = blockIdx.x; tb < n_sched && alive; tb += 32LL * gridDim.x) {
        const long long t = tb + (long long)lane * gridDim.x;
        long long ob = 0;
        int os = 0, nr = 0;  // (a tile that turned out empty would still be consumed, and store nothing)
        TcTile tl;
        if (t < n_sched && tc_tile<WORDS>(job, t, tiles_per_seg, &tl, s_len, s_bud, s_pref, nseq_dense, &cursor))
          ob = tl.out_base + tl.row0 * tl.out_stride, os = (int)tl.out_stride, nr = tl.nrows;
        const long long left = (n_sched - tb + gridDim.x - 1) / gridDim.x;
        const int cnt = left < 32 ? (int)left : 32;
        for (int j = 0; j < cnt && alive; ++j) {
          const long long obj = __shfl_sync(0xFFFFFFFFu, ob, j);
          const int osj = __shfl_sync(0xFFFFFFFFu, os, j), nrj = __shfl_sync(0xFFFFFFFFu, nr, j);
          alive = epi_tile(obj, osj, nrj);
          if (alive) ++it;
        }
      }
    } else {
      for (long long t = blockIdx.x; t < n_sched; t += gridDim.x) {
        TcTile tl;
        if (!tc_tile<WORDS>(job, t, tiles_per_seg, &tl, s_len, s_bud, s_pref, nseq_dense, &cursor)) continue;
        if (!epi_tile(tl.out_base + tl.row0 * tl.out_stride, (int)tl.out_stride, tl.nrows)) break;
        ++it;
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
  if (tid == 0 && abort_flag) atomicAdd(&g_tc_error, 1);
  griddep_wait();  // no-op unless this kernel was launched programmatically behind another one
}

}  // namespace he
