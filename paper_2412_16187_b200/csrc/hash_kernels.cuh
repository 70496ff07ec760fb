// he_hash_keys and phase 1 of he_prefill_compress: Eq. 2 on many rows with CUDA-core fp32 FMAs.
// A CTA stages W (zero-padded to 32 or 64 columns) and a tile of 128 rows in shared memory as fp32; each warp owns
// 16 rows and each lane one (or two) hash bits, so a row's sign bits are packed by one warp ballot per code word.
#pragma once
#include "common.cuh"

namespace he {

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
  const void* x2;              // mode 0, tensor-core kernel only: a second range of rows2 rows with the same stride, hashed by
  long long rows2;             //   the same launch; its codes follow the first range's in `out`
  long long s0, s1, s2;        // modes 1, 2: element strides (batch, head, token)
  int heads, G, Hkv;           // heads = heads per sequence of this tensor
  long long Nmax;
  const int32_t* prompt_len;
  const int32_t* budget;
  int q_all;            // mode 2: hash the queries of every prompt token, not only of those that evict
  const void* w_image;  // optional: the tensor-core kernel's shared-memory image of W's three bf16 terms (build_w_image_kernel)
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
    const long long C = max(job.budget[s], 0);
    const long long N = clamp_len(job.prompt_len[s], job.Nmax, (int)min(C, 1LL));
    base = static_cast<const char*>(job.x) + (s * job.s0 + hh * job.s1) * es;
    stride = job.s2;
    r_end = N;
    if (job.mode == 1) {
      r_begin = 0;
      out_base = ((long long)s * job.Hkv + hh) * job.Nmax * WORDS;
      out_stride = WORDS;
    } else {
      r_begin = job.q_all ? 0 : (C < N ? C : N);  // queries of appended tokens are never read by Algorithm 1
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

}  // namespace he
