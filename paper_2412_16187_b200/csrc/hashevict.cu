// HashEvict eviction hot path for B200 (sm_100a): host side of the C ABI declared in include/hashevict.h.
//
// The kernels live in the .cuh files next to this one:
//   hash_kernels.cuh, hash_tc_kernels.cuh   Eq. 2 on many rows (he_hash_keys, phase 1 of he_prefill_compress)
//   decode_kernels.cuh, decode_sm_kernels.cuh   Algorithm 1 lines 1-5 (he_decode_step)
//   prefill_kernels.cuh, prefill_tc_kernels.cuh   the prompt-encoding replay and the K/V gather (phases 2, 3 of
//                                                 he_prefill_compress)
//
// Eq. 2 is evaluated in one of two ways. CUDA cores (fp32 rows, odd head sizes, small calls, the per-unit decode
// kernel): channels are cut into chunks of 32; a chunk's partial sum is an fmaf chain in ascending channel order
// starting from 0; the partial sums are added in ascending chunk order; the bit is (sum >= 0). Tensor cores (bf16
// rows in bulk, and the one-CTA-per-SM decode kernel): W as three bf16 terms whose sum is W exactly, every product
// exact, fp32 accumulation in the instruction's own order. Both stay far inside the tolerance of Eq. 2's contract (a
// bit may differ from exact arithmetic only where the exact projection is within 1e-5 * |x| * |w| of zero), but they
// are two roundings of the same sum: for such a borderline bit two paths may disagree with each other.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <utility>

#include "attend_kernels.cuh"
#include "common.cuh"
#include "decode_kernels.cuh"
#include "decode_sm_kernels.cuh"
#include "hash_kernels.cuh"
#include "hash_tc_kernels.cuh"
#include "hashevict.h"
#include "oneshot_kernels.cuh"
#include "prefill_kernels.cuh"
#include "prefill_tc_kernels.cuh"

using namespace he;

namespace {

thread_local char g_err[512] = "";
thread_local cudaEvent_t g_phase_events[5] = {};  // he_prefill_phase_events: recorded between the phases of a prefill call
thread_local bool g_phase_events_on = false;

void record_phase(int i, cudaStream_t st) {
  if (g_phase_events_on && g_phase_events[i] != nullptr) cudaEventRecord(g_phase_events[i], st);
}

int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

#define HE_CUDA_CHECK(expr)                                                                         \
  do {                                                                                              \
    cudaError_t e_ = (expr);                                                                        \
    if (e_ != cudaSuccess) return fail(HE_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e_)); \
  } while (0)

__global__ void reset_kernel(const he_config cfg, const he_cache ca) {
  const long long units = (long long)cfg.batch * cfg.n_kv_heads;
  const long long slots = units * cfg.max_budget;
  const int Wd = words_of(cfg.hash_bits);
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < slots; i += stride) {
    ca.pos[i] = -1;
    ca.scores[i] = 0.f;
    const int cb = packed_code_bytes(cfg);
    if (cb == 0) {
      for (int w = 0; w < Wd; ++w) ca.codes[i * Wd + w] = 0u;
    } else {
      for (int w = 0; w < cb; ++w) reinterpret_cast<uint8_t*>(ca.codes)[i * cb + w] = 0;
    }
    if (i < units) {
      ca.fill[i] = 0;
      ca.next_pos[i] = 0;
    }
  }
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_config(const he_config* cfg, bool need_cache_dims) {
  if (cfg == nullptr) return fail(HE_ERR_INVALID_ARG, "cfg is null");
  if (cfg->dtype != HE_DTYPE_F32 && cfg->dtype != HE_DTYPE_BF16) return fail(HE_ERR_INVALID_ARG, "dtype %d is not HE_DTYPE_F32/BF16", cfg->dtype);
  if (cfg->hash_bits < 1 || cfg->hash_bits > 64) return fail(HE_ERR_INVALID_ARG, "hash_bits %d outside [1, 64]", cfg->hash_bits);
  if (cfg->head_dim < 8 || cfg->head_dim % 8 != 0) return fail(HE_ERR_INVALID_ARG, "head_dim %d is not a positive multiple of 8", cfg->head_dim);
  if (cfg->head_dim > kMaxDim) return fail(HE_ERR_UNSUPPORTED, "head_dim %d > %d", cfg->head_dim, kMaxDim);
  if (!need_cache_dims) return HE_OK;
  if (cfg->batch < 1 || cfg->n_kv_heads < 1) return fail(HE_ERR_INVALID_ARG, "batch %d / n_kv_heads %d must be >= 1", cfg->batch, cfg->n_kv_heads);
  if (cfg->group_size < 1) return fail(HE_ERR_INVALID_ARG, "group_size %d must be >= 1", cfg->group_size);
  if (cfg->group_size > kMaxGroup) return fail(HE_ERR_UNSUPPORTED, "group_size %d > %d", cfg->group_size, kMaxGroup);
  if (cfg->max_budget < 4 || cfg->max_budget % 4 != 0) return fail(HE_ERR_INVALID_ARG, "max_budget %d is not a positive multiple of 4", cfg->max_budget);
  if (cfg->max_budget > (1 << kKeyIdxBits)) return fail(HE_ERR_UNSUPPORTED, "max_budget %d > 2^20", cfg->max_budget);
  if (cfg->n_sink < 0 || cfg->n_recent < 0) return fail(HE_ERR_INVALID_ARG, "n_sink / n_recent must be >= 0");
  if (const int cb = packed_code_bytes(*cfg)) {
    if (cb > 3) return fail(HE_ERR_UNSUPPORTED, "packed codes of %d bytes per slot (hash_bits %d): 1 to 3, or whole words", cb, cfg->hash_bits);
    if (((long long)cfg->max_budget * cb) % 16 != 0)
      return fail(HE_ERR_INVALID_ARG, "packed codes: max_budget %d x %d bytes must be a multiple of 16", cfg->max_budget, cb);
  }
  return HE_OK;
}

int check_cache(const he_cache* ca) {
  if (ca == nullptr) return fail(HE_ERR_INVALID_ARG, "cache is null");
  if (!ca->k_cache || !ca->v_cache || !ca->codes || !ca->scores || !ca->pos || !ca->budget || !ca->fill || !ca->next_pos || !ca->W)
    return fail(HE_ERR_INVALID_ARG, "cache has a null pointer");
  if (!aligned16(ca->k_cache) || !aligned16(ca->v_cache) || !aligned16(ca->codes) || !aligned16(ca->scores) || !aligned16(ca->pos))
    return fail(HE_ERR_INVALID_ARG, "cache arrays must be 16-byte aligned");
  return HE_OK;
}

// Budgets must lie in [1, max_budget]; the host can only check them when the caller gave a mirror.
int check_budget_mirror(const he_config* cfg, const he_cache* ca) {
  if (ca->budget_host == nullptr) return HE_OK;
  for (int s = 0; s < cfg->batch; ++s)
    if (ca->budget_host[s] < 1 || ca->budget_host[s] > cfg->max_budget)
      return fail(HE_ERR_INVALID_ARG, "budget %d of sequence %d outside [1, max_budget = %d]", ca->budget_host[s], s, cfg->max_budget);
  return HE_OK;
}

// Dynamic shared memory above the default limit needs a per-function opt-in; it is asked for once per
// (device, kernel) and again only if a larger size is needed.
template <typename K>
int set_smem(K kernel, size_t bytes) {
  // static + dynamic shared memory beyond 48 KB needs the opt-in, so ask whenever the sum could exceed it
  if (bytes <= 24 * 1024) return HE_OK;
  static std::mutex mu;
  static std::map<std::pair<int, const void*>, size_t> granted;
  int dev = 0;
  HE_CUDA_CHECK(cudaGetDevice(&dev));
  std::lock_guard<std::mutex> lock(mu);
  size_t& have = granted[std::make_pair(dev, reinterpret_cast<const void*>(kernel))];
  if (bytes > have) {
    HE_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
    have = bytes;
  }
  return HE_OK;
}

constexpr long long kSplitDecodeRows = 16384;  // new rows per step from which he_decode_step hashes them in bulk first

// Decode launches carry the programmatic-serialization attribute so that consecutive he_decode_step kernels of a
// stream (or of a captured graph) overlap their launch latency; set HE_DISABLE_PDL=1 to launch them plainly.
bool pdl_enabled() {
  static const bool on = [] {
    const char* e = getenv("HE_DISABLE_PDL");
    return !(e && e[0] == '1');
  }();
  return on;
}

// Environment switches are read once per process (ID separates the call sites' caches).
template <int ID>
bool env_flag_set(const char* name) {
  static const bool on = getenv(name) != nullptr;
  return on;
}

bool tc_enabled() {
  static const bool on = [] {
    const char* e = getenv("HE_DISABLE_TC");
    return !(e && e[0] == '1');
  }();
  return on;
}

int sm_count(int* out) {
  static int cached[64] = {};
  int dev = 0;
  HE_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return fail(HE_ERR_UNSUPPORTED, "device index %d", dev);
  if (cached[dev] == 0) HE_CUDA_CHECK(cudaDeviceGetAttribute(&cached[dev], cudaDevAttrMultiProcessorCount, dev));
  *out = cached[dev];
  return HE_OK;
}

// Tensor map of the rows to hash, as a 4-D bf16 tensor {channel, row or token, head, sequence} with a box of
// 64 channels x 128 rows and the 128-byte shared-memory swizzle. Returns false when the driver's encoder is not
// available or rejects the strides (the kernel then stages rows with cp.async instead).
bool encode_rows_tmap(const HashJob& job, long long max_rows_per_segment, int segments, CUtensorMap* out) {
  using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static EncodeFn encode = [] {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      fn = nullptr;
    return reinterpret_cast<EncodeFn>(fn);
  }();
  memset(out, 0, sizeof(*out));
  if (encode == nullptr || env_flag_set<2>("HE_DISABLE_TMA")) return false;
  cuuint64_t dims[4], strides[3];
  dims[0] = (cuuint64_t)job.d;
  if (job.mode == 0) {
    dims[1] = (cuuint64_t)job.rows;
    dims[2] = 1;
    dims[3] = 1;
    strides[0] = (cuuint64_t)job.row_stride * 2;
    strides[1] = strides[0] * dims[1];
    strides[2] = strides[1];
  } else {
    dims[1] = (cuuint64_t)max_rows_per_segment;
    dims[2] = (cuuint64_t)job.heads;
    dims[3] = (cuuint64_t)(segments / job.heads);
    strides[0] = (cuuint64_t)job.s2 * 2;
    strides[1] = (cuuint64_t)job.s1 * 2;
    strides[2] = (cuuint64_t)job.s0 * 2;
  }
  for (int i = 0; i < 3; ++i)
    if (strides[i] % 16 != 0 || strides[i] >= (1ull << 40)) return false;
  for (int i = 0; i < 4; ++i)
    if (dims[i] == 0 || dims[i] > (1ull << 32)) return false;
  const cuuint32_t box[4] = {64, (cuuint32_t)kTcRows, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUresult r = encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(job.x), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Eq. 2 on many rows. bf16 rows with d = 64 or 128 go to the tensor-core kernel once there are enough of them to
// pay for staging the split W per CTA; everything else runs on the CUDA-core kernel.
int launch_hash(const HashJob& job, long long max_rows_per_segment, int segments, cudaStream_t stream, bool* image_built = nullptr,
                bool pdl = false) {
  if (max_rows_per_segment <= 0 || segments <= 0) return HE_OK;
  const int Wd = words_of(job.b);
  const long long tiles = (max_rows_per_segment + kHashRows - 1) / kHashRows;
  // flat rows may come as two ranges (the decode step's query rows and key rows): one launch of the tensor-core kernel
  const bool two = job.mode == 0 && job.x2 != nullptr && job.rows2 > 0;
  const long long tiles2 = two ? (job.rows2 + kHashRows - 1) / kHashRows : 0;
  const bool tc = tc_enabled() && job.dtype == HE_DTYPE_BF16 && (job.d == 64 || job.d == 128) && (tiles + tiles2) * segments >= 64;
  if (two && !tc) {  // the CUDA-core kernel takes one range at a time
    HashJob j1 = job, j2 = job;
    j1.x2 = nullptr, j1.rows2 = 0;
    j2.x = job.x2, j2.rows = job.rows2, j2.out = job.out + job.rows * Wd, j2.x2 = nullptr, j2.rows2 = 0;
    if (int rc = launch_hash(j1, j1.rows, 1, stream, image_built, pdl)) return rc;
    return launch_hash(j2, j2.rows, 1, stream, image_built, true);
  }
  if (tc) {
    static_assert(kTcRows == kHashRows, "both kernels tile rows by 128");
    const int N = 32 * Wd, KH = job.d / 64;
    const size_t smem = 1024 + (size_t)3 * KH * N * 128 + (size_t)kTcStages * KH * kTcRows * 128;
    int sms = 0;
    if (int rc = sm_count(&sms)) return rc;
    const long long total = tiles * segments + tiles2;
    const unsigned grid = (unsigned)(total < sms ? total : sms);
    alignas(64) CUtensorMap tmap, tmap2;
    bool tma = encode_rows_tmap(job, max_rows_per_segment, segments, &tmap);
    if (two) {
      HashJob j2 = job;
      j2.x = job.x2, j2.rows = job.rows2;
      tma = encode_rows_tmap(j2, j2.rows, 1, &tmap2) && tma;
    } else {
      tmap2 = tmap;
    }
    if (job.w_image != nullptr && (image_built == nullptr || !*image_built)) {  // scratch of kWImageBytes: filled once per call
      build_w_image_kernel<<<(job.d * N + 255) / 256, 256, 0, stream>>>(job.W, job.d, job.b, N,
                                                                       static_cast<unsigned char*>(const_cast<void*>(job.w_image)));
      HE_CUDA_CHECK(cudaGetLastError());
      if (image_built != nullptr) *image_built = true;
    }
    auto go = [&](auto kernel) -> int {
      if (int rc = set_smem(kernel, smem)) return rc;
      cudaLaunchConfig_t lc{};
      lc.gridDim = dim3(grid);
      lc.blockDim = dim3(kTcThreads);
      lc.dynamicSmemBytes = smem;
      lc.stream = stream;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[0].val.programmaticStreamSerializationAllowed = 1;
      lc.attrs = attr;
      lc.numAttrs = (pdl && pdl_enabled()) ? 1 : 0;
      HE_CUDA_CHECK(cudaLaunchKernelEx(&lc, kernel, job, total, tiles, tmap, tmap2));
      return HE_OK;
    };
    int rc;
    if (Wd == 1) rc = tma ? go(hash_rows_tc_kernel<1, true>) : go(hash_rows_tc_kernel<1, false>);
    else rc = tma ? go(hash_rows_tc_kernel<2, true>) : go(hash_rows_tc_kernel<2, false>);
    if (rc) return rc;
    HE_CUDA_CHECK(cudaGetLastError());
    return HE_OK;
  }
  const size_t smem = ((size_t)job.d * 32 * Wd + (size_t)kHashRows * job.d) * sizeof(float);
  if (tiles > 0x7FFFFFFFLL || segments > 65535) return fail(HE_ERR_UNSUPPORTED, "hash grid too large (%lld x %d)", tiles, segments);
  dim3 grid((unsigned)tiles, (unsigned)segments);
  if (Wd == 1) {
    if (int rc = set_smem(hash_rows_kernel<1>, smem)) return rc;
    hash_rows_kernel<1><<<grid, kHashThreads, smem, stream>>>(job);
  } else {
    if (int rc = set_smem(hash_rows_kernel<2>, smem)) return rc;
    hash_rows_kernel<2><<<grid, kHashThreads, smem, stream>>>(job);
  }
  HE_CUDA_CHECK(cudaGetLastError());
  return HE_OK;
}

template <int WORDS, int GT, int NT, bool PRE, bool PACKED = false>
int launch_decode_one(const DecodeArgs& a, size_t smem, dim3 grid, cudaStream_t stream) {
  if (int rc = set_smem(decode_step_kernel<WORDS, GT, NT, PRE, PACKED>, smem)) return rc;
  cudaLaunchConfig_t lc{};
  lc.gridDim = grid;
  lc.blockDim = dim3(NT);
  lc.dynamicSmemBytes = smem;
  lc.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = pdl_enabled() ? 1 : 0;
  HE_CUDA_CHECK(cudaLaunchKernelEx(&lc, decode_step_kernel<WORDS, GT, NT, PRE, PACKED>, a));
  return HE_OK;
}

template <int WORDS, int GT, bool PACKED>
int launch_decode_nt(const DecodeArgs& a, int nt, size_t smem, dim3 grid, cudaStream_t stream) {
  if (a.new_codes != nullptr) {
    if (nt == 256) return launch_decode_one<WORDS, GT, 256, true, PACKED>(a, smem, grid, stream);
    if (nt == 512) return launch_decode_one<WORDS, GT, 512, true, PACKED>(a, smem, grid, stream);
    return launch_decode_one<WORDS, GT, 1024, true, PACKED>(a, smem, grid, stream);
  }
  if (nt == 256) return launch_decode_one<WORDS, GT, 256, false, PACKED>(a, smem, grid, stream);
  if (nt == 512) return launch_decode_one<WORDS, GT, 512, false, PACKED>(a, smem, grid, stream);
  return launch_decode_one<WORDS, GT, 1024, false, PACKED>(a, smem, grid, stream);
}

template <int WORDS, bool PACKED = false>
int launch_decode_g(const DecodeArgs& a, int nt, size_t smem, dim3 grid, cudaStream_t stream) {
  switch (a.cfg.group_size) {
    case 1: return launch_decode_nt<WORDS, 1, PACKED>(a, nt, smem, grid, stream);
    case 4: return launch_decode_nt<WORDS, 4, PACKED>(a, nt, smem, grid, stream);
    default: return launch_decode_nt<WORDS, 0, PACKED>(a, nt, smem, grid, stream);
  }
}

// One CTA per SM (decode_sm_kernels.cuh), for HE_FLAG_EARLY_INPUTS: q, k, v are read and hashed before the wait.
template <int WORDS, int GT, bool MMA>
int launch_decode_sm_one(const DecodeArgs& a, unsigned grid, cudaStream_t stream) {
  const size_t smem = sm_layout(a.cfg.head_dim, WORDS, esize_of(a.cfg.dtype), MMA).total;
  if (int rc = set_smem(decode_step_sm_kernel<WORDS, GT, MMA>, smem)) return rc;
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3(grid);
  lc.blockDim = dim3(kSmThreads);
  lc.dynamicSmemBytes = smem;
  lc.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = pdl_enabled() ? 1 : 0;
  HE_CUDA_CHECK(cudaLaunchKernelEx(&lc, decode_step_sm_kernel<WORDS, GT, MMA>, a));
  return HE_OK;
}

template <int WORDS, int GT>
int launch_decode_sm_g(const DecodeArgs& a, bool mma, unsigned grid, cudaStream_t stream) {
  return mma ? launch_decode_sm_one<WORDS, GT, true>(a, grid, stream) : launch_decode_sm_one<WORDS, GT, false>(a, grid, stream);
}

template <int WORDS>
int launch_decode_sm(const DecodeArgs& a, bool mma, unsigned grid, cudaStream_t stream) {
  switch (a.cfg.group_size) {
    case 1: return launch_decode_sm_g<WORDS, 1>(a, mma, grid, stream);
    case 4: return launch_decode_sm_g<WORDS, 4>(a, mma, grid, stream);
    default: return launch_decode_sm_g<WORDS, 0>(a, mma, grid, stream);
  }
}

// Sequences ordered by budget, largest first (ties by index), each with its budget, for the unit schedule of the
// one-CTA-per-SM decode kernel: word = sequence << 21 | budget. The caller's budget mirror is hashed on every call
// and sorted again only when its contents changed.
struct SchedCache {
  uint64_t hash = 0;
  int n = -1;
  int cmax = 0;
  uint32_t sched[kMaxBudgetVals];
};
const uint32_t* sched_of(const int32_t* budget_host, int n, int cmax) {
  thread_local SchedCache c;
  uint64_t h = 1469598103934665603ull;
  for (int i = 0; i < n; ++i) h = (h ^ (uint32_t)budget_host[i]) * 1099511628211ull;
  if (c.n != n || c.hash != h || c.cmax != cmax) {
    uint16_t order[kMaxBudgetVals];
    for (int i = 0; i < n; ++i) order[i] = (uint16_t)i;
    std::stable_sort(order, order + n, [&](uint16_t x, uint16_t y) { return budget_host[x] > budget_host[y]; });
    for (int i = 0; i < n; ++i) {
      const int cb = budget_host[order[i]];
      c.sched[i] = ((uint32_t)order[i] << kSmSchedShift) | (uint32_t)(cb < 0 ? 0 : (cb > cmax ? cmax : cb));
    }
    c.n = n;
    c.hash = h;
    c.cmax = cmax;
  }
  return c.sched;
}

template <int WORDS, int GT>
int launch_replay_smem(const ReplayArgs& a, long long units, cudaStream_t stream) {
  const size_t smem = (size_t)a.cfg.max_budget * (WORDS + 1) * 4;
  if (smem > 200 * 1024) return fail(HE_ERR_UNSUPPORTED, "max_budget %d does not fit the replay kernel's shared memory", a.cfg.max_budget);
  int nt = 256;
  if (a.cfg.max_budget > 4096) nt = 512;
  if (a.cfg.max_budget > 16384) nt = 1024;
  if (int rc = set_smem(prefill_replay_smem_kernel<WORDS, GT>, smem)) return rc;
  prefill_replay_smem_kernel<WORDS, GT><<<(unsigned)units, nt, smem, stream>>>(a);
  HE_CUDA_CHECK(cudaGetLastError());
  return HE_OK;
}

// The register kernel is persistent: as many CTAs as fit the GPU at once, each claiming units from the schedule.
template <int WORDS, int GT, int SPT, int NT>
int launch_replay_reg_one(const ReplayArgs& a, long long units, cudaStream_t stream) {
  const size_t smem = (size_t)a.cfg.max_budget * 4;
  if (int rc = set_smem(prefill_replay_reg_kernel<WORDS, GT, SPT, NT>, smem)) return rc;
  static int per_sm[64] = {};
  int dev = 0, sms = 0;
  HE_CUDA_CHECK(cudaGetDevice(&dev));
  if (int rc = sm_count(&sms)) return rc;
  if (per_sm[dev] == 0) {
    int n = 0;
    HE_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, prefill_replay_reg_kernel<WORDS, GT, SPT, NT>, NT, smem));
    per_sm[dev] = n > 0 ? n : 1;
  }
  const int nbins = sms < kMaxBins ? sms : kMaxBins;
  prefill_schedule_kernel<<<1, kSchedThreads, 0, stream>>>(a.cfg, a.ca.budget, a.prompt_len, nbins, a.sched, 0);
  HE_CUDA_CHECK(cudaGetLastError());
  long long grid = (long long)sms * per_sm[dev];
  if (grid > units) grid = units;
  prefill_replay_reg_kernel<WORDS, GT, SPT, NT><<<(unsigned)grid, NT, smem, stream>>>(a);
  HE_CUDA_CHECK(cudaGetLastError());
  return HE_OK;
}

// Smallest (threads x slots-per-thread) tile of the register kernel that holds max_budget slots.
template <int WORDS, int GT>
int launch_replay_reg(const ReplayArgs& a, long long units, cudaStream_t stream) {
  const int c = a.cfg.max_budget;
  if (c <= 256 * 4) return launch_replay_reg_one<WORDS, GT, 4, 256>(a, units, stream);
  if (c <= 256 * 8) return launch_replay_reg_one<WORDS, GT, 8, 256>(a, units, stream);
  if (c <= 256 * 16) return launch_replay_reg_one<WORDS, GT, 16, 256>(a, units, stream);
  if (c <= 512 * 16) return launch_replay_reg_one<WORDS, GT, 16, 512>(a, units, stream);
  if (c <= 512 * 20) return launch_replay_reg_one<WORDS, GT, 20, 512>(a, units, stream);
  if (c <= 512 * 24) return launch_replay_reg_one<WORDS, GT, 24, 512>(a, units, stream);
  if (c <= 1024 * 16) return launch_replay_reg_one<WORDS, GT, 16, 1024>(a, units, stream);
  return launch_replay_smem<WORDS, GT>(a, units, stream);
}

// Tensor-core replay: one persistent CTA per SM, for budgets up to 12288 slots. Up to 4096 slots the unit's tables sit in
// shared memory, beyond that they are the cache's own arrays.
template <int WORDS, bool GLOBAL_TABLE, bool FP8, bool PROT = false, bool RUNS = true>
int launch_replay_tc_one(const ReplayArgs& a0, long long units, cudaStream_t stream) {
  ReplayArgs a = a0;
  a.smem_slots = (a.cfg.max_budget + kRtTile - 1) / kRtTile * kRtTile;
  const size_t smem = rt_layout(WORDS, a.smem_slots, a.cfg.group_size, !GLOBAL_TABLE, FP8).total;
  if (int rc = set_smem(prefill_replay_tc_kernel<WORDS, GLOBAL_TABLE, FP8, PROT, RUNS>, smem)) return rc;
  int sms = 0;
  if (int rc = sm_count(&sms)) return rc;
  const int nbins = sms < kMaxBins ? sms : kMaxBins;
  // a step of this kernel costs about 400 cycles of resolver time plus 0.06 cycles per slot of tile work
  prefill_schedule_kernel<<<1, kSchedThreads, 0, stream>>>(a.cfg, a.ca.budget, a.prompt_len, nbins, a.sched, 6700);
  HE_CUDA_CHECK(cudaGetLastError());
  const long long grid = units < sms ? units : sms;
  prefill_replay_tc_kernel<WORDS, GLOBAL_TABLE, FP8, PROT, RUNS><<<(unsigned)grid, kRtThreads, smem, stream>>>(a);
  HE_CUDA_CHECK(cudaGetLastError());
  return HE_OK;
}

// 8-bit operands when the group's code sum fits e5m2 exactly (group sizes up to 7); HE_TC_REPLAY_BF16=1 keeps bf16.
template <int WORDS, bool GLOBAL_TABLE>
int launch_replay_tc(const ReplayArgs& a, long long units, cudaStream_t stream) {
  static const bool bf16_forced = [] {
    const char* e = getenv("HE_TC_REPLAY_BF16");
    return e && e[0] == '1';
  }();
  const bool fp8 = a.cfg.group_size <= 7 && !bf16_forced;
  if (a.cfg.n_sink > 0 || a.cfg.n_recent > 0)  // protected windows
    return fp8 ? launch_replay_tc_one<WORDS, GLOBAL_TABLE, true, true>(a, units, stream)
               : launch_replay_tc_one<WORDS, GLOBAL_TABLE, false, true>(a, units, stream);
  if (fp8) {
    // no unit of such a launch can use the run-based resolver loop (every table keeps its tiles' second-largest keys)
    if (!GLOBAL_TABLE && a.cfg.max_budget <= kRtSecondMaxTiles * kRtTile)
      return launch_replay_tc_one<WORDS, false, true, false, false>(a, units, stream);
    return launch_replay_tc_one<WORDS, GLOBAL_TABLE, true>(a, units, stream);
  }
  return launch_replay_tc_one<WORDS, GLOBAL_TABLE, false>(a, units, stream);
}

// HE_TC_REPLAY=0 keeps the replay on the CUDA-core kernels, =1 sends every eligible shape to the tensor-core kernel.
// Unset: the tensor-core kernel runs one unit per SM at about 400 cycles per step whatever the budget, the register
// kernel several units per SM at a cost that grows with the budget; measured on B200 (512 units, b = 64, G = 4) they
// cross between 1024 and 1280 slots, and with no more units than SMs already around 512 slots.
int tc_replay_mode() {
  static const int mode = [] {
    const char* e = getenv("HE_TC_REPLAY");
    if (!tc_enabled() || (e && e[0] == '0')) return 0;
    return (e && e[0] == '1') ? 2 : 1;
  }();
  return mode;
}

template <int WORDS>
int launch_replay(const ReplayArgs& a, long long units, cudaStream_t stream) {
  const int mode = tc_replay_mode();
  int sms = 0;
  if (int rc = sm_count(&sms)) return rc;
  const int min_budget = units <= sms ? 512 : 1152;
  bool tc_ok = mode != 0 && a.cfg.max_budget <= kRtMaxSlotsGlobal && (mode == 2 || a.cfg.max_budget >= min_budget);
  // beyond 4096 slots the tensor-core kernel keeps its working table in the cache's own code array: word layout only
  if (a.cfg.max_budget > kRtMaxSlots && packed_code_bytes(a.cfg) != 0) tc_ok = false;
  if (tc_ok && (a.cfg.n_sink > 0 || a.cfg.n_recent > 0)) {
    // protected windows: every budget must leave an eligible slot at every step (n_sink + n_recent < C), which the host
    // can only check on the caller's mirror of the budgets; with the tables in global memory the kernel tracks the
    // recent tokens in a 32-entry ring
    tc_ok = a.cfg.n_recent <= (a.cfg.max_budget <= kRtMaxSlots ? kRtRows - 1 : 32) && a.ca.budget_host != nullptr;
    for (int s = 0; tc_ok && s < a.cfg.batch; ++s) tc_ok = a.ca.budget_host[s] > a.cfg.n_sink + a.cfg.n_recent;
  }
  if (tc_ok)
    return a.cfg.max_budget <= kRtMaxSlots ? launch_replay_tc<WORDS, false>(a, units, stream)
                                           : launch_replay_tc<WORDS, true>(a, units, stream);
  switch (a.cfg.group_size) {
    case 1: return launch_replay_reg<WORDS, 1>(a, units, stream);
    case 4: return launch_replay_reg<WORDS, 4>(a, units, stream);
    default: return launch_replay_smem<WORDS, 0>(a, units, stream);
  }
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Scratch of he_prefill_compress_noalloc: part of the device image, so no allocation is ever needed for it.
// In host code this name is only a handle for the runtime's symbol calls, never a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[HE_NOALLOC_SCRATCH_BYTES];

}  // namespace

extern "C" {

const char* he_last_error(void) { return g_err; }

int he_prefill_phase_events(void* const* events) {
  g_phase_events_on = events != nullptr;
  for (int i = 0; i < 5; ++i) g_phase_events[i] = events != nullptr ? static_cast<cudaEvent_t>(events[i]) : nullptr;
  return HE_OK;
}

int he_device_error_count(void) {
  int n = 0;
  if (cudaMemcpyFromSymbol(&n, he::g_tc_error, sizeof(int)) != cudaSuccess) return -1;
  return n;
}

int he_hash_keys(const he_config* cfg, const void* x, int64_t rows, int64_t row_stride_elems, const float* W,
                 uint32_t* codes_out, void* stream) {
  if (int rc = check_config(cfg, false)) return rc;
  if (rows < 0) return fail(HE_ERR_INVALID_ARG, "rows %lld < 0", (long long)rows);
  if (rows == 0) return HE_OK;
  if (!x || !W || !codes_out) return fail(HE_ERR_INVALID_ARG, "x, W or codes_out is null");
  const int es = esize_of(cfg->dtype);
  if (row_stride_elems < cfg->head_dim || (row_stride_elems * es) % 16 != 0 || !aligned16(x))
    return fail(HE_ERR_INVALID_ARG, "rows of x must be 16-byte aligned with a stride >= head_dim");
  HashJob job{};
  job.x = x;
  job.W = W;
  job.out = codes_out;
  job.mode = 0;
  job.dtype = cfg->dtype;
  job.d = cfg->head_dim;
  job.b = cfg->hash_bits;
  job.rows = rows;
  job.row_stride = row_stride_elems;
  return launch_hash(job, rows, 1, static_cast<cudaStream_t>(stream));
}

int he_decode_step(const he_config* cfg, const he_cache* cache, const void* q, const void* k, const void* v,
                   int32_t* victim_out, int32_t* evicted_pos_out, uint32_t* qcodes_out, void* stream) {
  if (int rc = check_config(cfg, true)) return rc;
  if (int rc = check_cache(cache)) return rc;
  if (!q || !k || !v || !victim_out) return fail(HE_ERR_INVALID_ARG, "q, k, v or victim_out is null");
  if (!aligned16(q) || !aligned16(k) || !aligned16(v)) return fail(HE_ERR_INVALID_ARG, "q, k, v must be 16-byte aligned");
  if (int rc = check_budget_mirror(cfg, cache)) return rc;
  const int Wd = words_of(cfg->hash_bits);
  const int cb = packed_code_bytes(*cfg);  // 1..3 bytes per slot, or 0: word layout
  const long long nvec = cb ? ((long long)cfg->max_budget * cb + 15) / 16 : ((long long)cfg->max_budget * Wd + 3) / 4;
  const size_t smem = (size_t)nvec * 16;
  if (smem > 200 * 1024) return fail(HE_ERR_UNSUPPORTED, "max_budget %d with %d code words does not fit the decode kernel's shared memory", cfg->max_budget, Wd);
  int nt = 256;
  if (nvec > 2048) nt = 512;
  if (nvec > 4096) nt = 1024;
  if (cb) nt = cfg->max_budget <= 4096 ? 256 : (cfg->max_budget <= 16384 ? 512 : 1024);
  if (!cb && nvec > 1024LL * kVecsPerThread)
    return fail(HE_ERR_UNSUPPORTED, "max_budget %d with %d code words exceeds the decode kernel's %d vectors", cfg->max_budget, Wd,
                1024 * kVecsPerThread);
  if (cfg->batch > 65535) return fail(HE_ERR_UNSUPPORTED, "batch %d > 65535 in one decode call", cfg->batch);
  if ((long long)cfg->batch * cfg->n_kv_heads * cfg->max_budget * Wd > 0x7FFFFFFFLL * 16)
    return fail(HE_ERR_UNSUPPORTED, "cache too large for one decode call");
  DecodeArgs a;
  a.cfg = *cfg;
  a.ca = *cache;
  a.q = q;
  a.k = k;
  a.v = v;
  a.victim_out = victim_out;
  a.evicted_pos_out = evicted_pos_out;
  a.qcodes_out = qcodes_out;
  a.n_budget_vals = 0;
  a.n_sched = 0;
  a.new_codes = nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // Large batches: hash the step's new rows with the bulk projection kernels (tensor cores for bf16) into the
  // caller's scratch, so the per-unit kernel only scans. Small batches keep the single fused kernel.
  const long long units_ll = (long long)cfg->batch * cfg->n_kv_heads;
  // HE_FLAG_EARLY_INPUTS: while the units fit four per SM-wide CTA, the one-CTA-per-SM kernel hashes the step's rows
  // before its wait. It serves whole-chunk head sizes with the word layout of the code table; larger batches keep the
  // per-unit kernels (many waves of small CTAs hide their own latencies).
  int sms = 0;
  if (int rc = sm_count(&sms)) return rc;
  const bool early = cb == 0 && cfg->head_dim % kChunk == 0 && (cfg->flags & HE_FLAG_EARLY_INPUTS) != 0 &&
                     units_ll <= (long long)kSmUnits * sms && !env_flag_set<0>("HE_DISABLE_EARLY_DECODE");
  if (early) {
    if (cache->budget_host != nullptr && cfg->batch <= kMaxBudgetVals) {
      a.n_sched = cfg->batch;
      memcpy(a.sched, sched_of(cache->budget_host, cfg->batch, cfg->max_budget), sizeof(uint32_t) * (size_t)cfg->batch);
    }
    const unsigned g = (unsigned)(units_ll < sms ? units_ll : sms);
    const bool mma = tc_enabled() && cfg->dtype == HE_DTYPE_BF16 && cfg->head_dim <= 128;
    return Wd == 1 ? launch_decode_sm<1>(a, mma, g, st) : launch_decode_sm<2>(a, mma, g, st);
  }
  if (cache->step_scratch != nullptr && units_ll * (cfg->group_size + 1) >= kSplitDecodeRows &&
      !env_flag_set<1>("HE_DISABLE_SPLIT_DECODE")) {
    HashJob job{};
    job.W = cache->W;
    job.mode = 0;
    job.dtype = cfg->dtype;
    job.d = cfg->head_dim;
    job.b = cfg->hash_bits;
    job.row_stride = cfg->head_dim;
    job.w_image = reinterpret_cast<char*>(cache->step_scratch) +
                  align_up((size_t)units_ll * (cfg->group_size + 1) * Wd * 4, 256);
    // the query rows and the key rows go through one launch; the key codes follow the query codes in the scratch
    job.x = q;
    job.rows = units_ll * cfg->group_size;
    job.x2 = k;
    job.rows2 = units_ll;
    job.out = cache->step_scratch;
    bool image_built = false;
    if (int rc = launch_hash(job, job.rows, 1, st, &image_built)) return rc;
    a.new_codes = cache->step_scratch;
  }
  if (cache->budget_host != nullptr && cfg->batch <= kMaxBudgetVals) {
    // budgets travel in the kernel parameters, so the code-table copy can start without a dependent device read
    a.n_budget_vals = cfg->batch;
    memcpy(a.budget_vals, cache->budget_host, sizeof(int32_t) * (size_t)cfg->batch);
  }
  const dim3 grid((unsigned)cfg->n_kv_heads, (unsigned)cfg->batch);
  if (cb) return launch_decode_g<1, true>(a, nt, smem, grid, st);
  return Wd == 1 ? launch_decode_g<1>(a, nt, smem, grid, st) : launch_decode_g<2>(a, nt, smem, grid, st);
}

size_t he_workspace_bytes(const he_config* cfg, int32_t max_prompt_len) {
  if (check_config(cfg, true) != HE_OK || max_prompt_len < 0) return 0;
  const size_t units = (size_t)cfg->batch * cfg->n_kv_heads;
  const size_t Wd = words_of(cfg->hash_bits);
  const size_t kbytes = align_up(units * (size_t)max_prompt_len * Wd * 4, 256);
  const size_t qbytes = align_up(units * (size_t)max_prompt_len * cfg->group_size * Wd * 4, 256);
  return kbytes + qbytes + align_up(sched_words((long long)units) * 4, 256) + align_up(kWImageBytes, 256) + 256;
}

size_t he_oneshot_workspace_bytes(const he_config* cfg, int32_t max_prompt_len) {
  const size_t base = he_workspace_bytes(cfg, max_prompt_len);
  if (base == 0) return 0;
  const size_t tokens = (size_t)cfg->batch * cfg->n_kv_heads * (size_t)max_prompt_len;
  return base + align_up(tokens * 4, 256) + align_up(tokens * 8, 256);
}

}  // extern "C"

namespace {

// Shared body of he_prefill_compress (oneshot = false: Algorithm 1 replayed over the prompt) and he_prefill_oneshot
// (oneshot = true: the averaged-Hamming ranking of Appendix C): validation, Eq. 2 on the prompt's keys and queries,
// the selection kernel(s), the gather of the surviving K / V rows.
int prefill_impl(int variant /* 0: Algorithm 1, 1: averaged Hamming, 2: L2 norm */, const he_config* cfg, const he_cache* cache, const void* q, const void* k, const void* v,
                 const int64_t q_strides[3], const int64_t kv_strides[3], const int32_t* prompt_len, int32_t max_prompt_len,
                 void* workspace, size_t workspace_bytes, void* rank_out, void* stream) {
  const bool oneshot = variant != 0;
  if (variant == 2) q = k, q_strides = kv_strides;  // no queries in this policy: only the checks below look at them
  if (int rc = check_config(cfg, true)) return rc;
  if (int rc = check_cache(cache)) return rc;
  if (!q || !k || !v || !q_strides || !kv_strides || !prompt_len || !workspace)
    return fail(HE_ERR_INVALID_ARG, "q, k, v, strides, prompt_len or workspace is null");
  if (max_prompt_len < 0) return fail(HE_ERR_INVALID_ARG, "max_prompt_len %d < 0", max_prompt_len);
  if (int rc = check_budget_mirror(cfg, cache)) return rc;
  const int es = esize_of(cfg->dtype);
  for (int i = 0; i < 3; ++i)
    if ((q_strides[i] * es) % 16 != 0 || (kv_strides[i] * es) % 16 != 0)
      return fail(HE_ERR_INVALID_ARG, "strides must keep every row 16-byte aligned");
  if (!aligned16(q) || !aligned16(k) || !aligned16(v)) return fail(HE_ERR_INVALID_ARG, "q, k, v must be 16-byte aligned");
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return fail(HE_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
  const size_t need = oneshot ? he_oneshot_workspace_bytes(cfg, max_prompt_len) : he_workspace_bytes(cfg, max_prompt_len);
  if (workspace_bytes < need) return fail(HE_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, need);
  if (oneshot && max_prompt_len > 32768) return fail(HE_ERR_UNSUPPORTED, "one-shot ranking: max_prompt_len %d > 32768", max_prompt_len);

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const long long units = (long long)cfg->batch * cfg->n_kv_heads;
  const int Wd = words_of(cfg->hash_bits), G = cfg->group_size;
  uint32_t* kcodes = static_cast<uint32_t*>(workspace);
  uint32_t* qcodes = reinterpret_cast<uint32_t*>(static_cast<char*>(workspace) +
                                                 align_up((size_t)units * max_prompt_len * Wd * 4, 256));

  bool image_built = false;
  record_phase(0, st);
  // phase 1: Eq. 2 on every prompt key and on the queries of the tokens that will evict
  HashJob job{};
  job.w_image = static_cast<char*>(workspace) + align_up((size_t)units * max_prompt_len * Wd * 4, 256) +
                align_up((size_t)units * max_prompt_len * G * Wd * 4, 256) + align_up(sched_words(units) * 4, 256);
  job.W = cache->W;
  job.dtype = cfg->dtype;
  job.d = cfg->head_dim;
  job.b = cfg->hash_bits;
  job.Hkv = cfg->n_kv_heads;
  job.G = G;
  job.Nmax = max_prompt_len;
  job.prompt_len = prompt_len;
  job.budget = cache->budget;
  job.x = k;
  job.out = kcodes;
  job.mode = 1;
  job.heads = cfg->n_kv_heads;
  job.s0 = kv_strides[0];
  job.s1 = kv_strides[1];
  job.s2 = kv_strides[2];
  if (int rc = launch_hash(job, max_prompt_len, (int)units, st, &image_built)) return rc;
  record_phase(1, st);
  if (variant != 2) {
  job.x = q;
  job.out = qcodes;
  job.mode = 2;
  job.q_all = oneshot ? 1 : 0;  // the ranking reads the queries of all later tokens, Algorithm 1 only those that evict
  job.heads = cfg->n_kv_heads * G;
  job.s0 = q_strides[0];
  job.s1 = q_strides[1];
  job.s2 = q_strides[2];
  if (int rc = launch_hash(job, max_prompt_len, (int)units * G, st, &image_built)) return rc;
  }

  record_phase(2, st);
  // phase 2: the sequential replay of Algorithm 1 over the prompt, one CTA per unit
  int32_t* sched = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(qcodes) +
                                              align_up((size_t)units * max_prompt_len * G * Wd * 4, 256));
  if (oneshot) {
    if (units > 0x7FFFFFFF) return fail(HE_ERR_UNSUPPORTED, "too many units");
    char* extra = static_cast<char*>(workspace) + he_workspace_bytes(cfg, max_prompt_len);
    OneshotArgs oa{*cfg, *cache, kcodes, qcodes, prompt_len, max_prompt_len, reinterpret_cast<int32_t*>(extra),
                   reinterpret_cast<unsigned long long*>(extra + align_up((size_t)units * max_prompt_len * 4, 256)),
                   variant == 1 ? static_cast<long long*>(rank_out) : nullptr};
    if (variant == 2) {
      if (units > 65535) return fail(HE_ERR_UNSUPPORTED, "more than 65535 units in one prefill call");
      NormArgs na{*cfg, k, kv_strides[0], kv_strides[1], kv_strides[2], prompt_len, max_prompt_len, oa.sums, static_cast<float*>(rank_out)};
      if (max_prompt_len > 0)
        key_norms_kernel<<<dim3((unsigned)((max_prompt_len + kOneshotThreads - 1) / kOneshotThreads), (unsigned)units), kOneshotThreads, 0, st>>>(na);
      HE_CUDA_CHECK(cudaGetLastError());
      if (Wd == 1) oneshot_rank_kernel<1, 1><<<(unsigned)units, kOneshotThreads, 0, st>>>(oa);
      else oneshot_rank_kernel<2, 1><<<(unsigned)units, kOneshotThreads, 0, st>>>(oa);
    } else {
      if (Wd == 1) oneshot_rank_kernel<1, 0><<<(unsigned)units, kOneshotThreads, 0, st>>>(oa);
      else oneshot_rank_kernel<2, 0><<<(unsigned)units, kOneshotThreads, 0, st>>>(oa);
    }
    HE_CUDA_CHECK(cudaGetLastError());
  } else {
    ReplayArgs ra{*cfg, *cache, kcodes, qcodes, prompt_len, max_prompt_len, cfg->max_budget, sched};
    if (int rc = (Wd == 1 ? launch_replay<1>(ra, units, st) : launch_replay<2>(ra, units, st))) return rc;
  }

  record_phase(3, st);
  // phase 3: surviving K / V rows into their slots
  GatherArgs ga{*cfg, *cache, k, v, kv_strides[0], kv_strides[1], kv_strides[2], max_prompt_len};
  const int cpr = cfg->head_dim * es / 16;
  if (units > 65535) return fail(HE_ERR_UNSUPPORTED, "more than 65535 units in one prefill call");
  if (cpr <= kGatherThreads && (cpr & (cpr - 1)) == 0) {  // rows of a power-of-two number of 16-byte chunks
    int lg = 0;
    while ((1 << lg) < cpr) ++lg;
    const int rows_per_cta = (kGatherThreads >> lg) * kGatherRows;
    const long long gx = ((long long)cfg->max_budget + rows_per_cta - 1) / rows_per_cta;
    prefill_gather_rows_kernel<<<dim3((unsigned)gx, (unsigned)units), kGatherThreads, 0, st>>>(ga, lg);
  } else {
    const long long per_unit = 2LL * cfg->max_budget * cpr;
    const long long gx = (per_unit + kGatherThreads * kGatherUnroll - 1) / (kGatherThreads * kGatherUnroll);
    prefill_gather_kernel<<<dim3((unsigned)gx, (unsigned)units), kGatherThreads, 0, st>>>(ga);
  }
  HE_CUDA_CHECK(cudaGetLastError());
  record_phase(4, st);
  return HE_OK;
}

}  // namespace

extern "C" {

int he_prefill_compress(const he_config* cfg, const he_cache* cache, const void* q, const void* k, const void* v,
                        const int64_t q_strides[3], const int64_t kv_strides[3], const int32_t* prompt_len,
                        int32_t max_prompt_len, void* workspace, size_t workspace_bytes, void* stream) {
  return prefill_impl(0, cfg, cache, q, k, v, q_strides, kv_strides, prompt_len, max_prompt_len, workspace, workspace_bytes,
                      nullptr, stream);
}

int he_prefill_oneshot(const he_config* cfg, const he_cache* cache, const void* q, const void* k, const void* v,
                       const int64_t q_strides[3], const int64_t kv_strides[3], const int32_t* prompt_len,
                       int32_t max_prompt_len, void* workspace, size_t workspace_bytes, long long* sums_out, void* stream) {
  return prefill_impl(1, cfg, cache, q, k, v, q_strides, kv_strides, prompt_len, max_prompt_len, workspace, workspace_bytes,
                      sums_out, stream);
}

int he_prefill_oneshot_l2(const he_config* cfg, const he_cache* cache, const void* k, const void* v, const int64_t kv_strides[3],
                          const int32_t* prompt_len, int32_t max_prompt_len, void* workspace, size_t workspace_bytes,
                          float* norms_out, void* stream) {
  return prefill_impl(2, cfg, cache, nullptr, k, v, nullptr, kv_strides, prompt_len, max_prompt_len, workspace, workspace_bytes,
                      norms_out, stream);
}

int he_prefill_compress_noalloc(const he_config* cfg, const he_cache* cache, const void* q, const void* k,
                                const void* v, const int64_t q_strides[3], const int64_t kv_strides[3],
                                const int32_t* prompt_len, int32_t max_prompt_len, void* stream) {
  if (int rc = check_config(cfg, true)) return rc;
  if (max_prompt_len < 0) return fail(HE_ERR_INVALID_ARG, "max_prompt_len %d < 0", max_prompt_len);
  const size_t need = he_workspace_bytes(cfg, max_prompt_len);
  if (need > HE_NOALLOC_SCRATCH_BYTES)
    return fail(HE_ERR_WORKSPACE, "prompt codes need %zu bytes, the built-in scratch holds %u; use he_prefill_compress with your own workspace",
                need, (unsigned)HE_NOALLOC_SCRATCH_BYTES);
  // device address of the built-in array, looked up once per device with that device current
  static std::mutex mu;
  static void* scratch_of_device[64] = {};
  int dev = 0;
  HE_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return fail(HE_ERR_UNSUPPORTED, "device index %d", dev);
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (scratch_of_device[dev] == nullptr) {
      void* p = nullptr;
      HE_CUDA_CHECK(cudaGetSymbolAddress(&p, g_noalloc_scratch));
      scratch_of_device[dev] = p;
    }
    scratch = scratch_of_device[dev];
  }
  return he_prefill_compress(cfg, cache, q, k, v, q_strides, kv_strides, prompt_len, max_prompt_len, scratch,
                             HE_NOALLOC_SCRATCH_BYTES, stream);
}

int he_attend(const he_config* cfg, const he_cache* cache, const void* q, float* out, void* stream) {
  if (int rc = check_config(cfg, true)) return rc;
  if (int rc = check_cache(cache)) return rc;
  if (!q || !out || !aligned16(q) || !aligned16(out)) return fail(HE_ERR_INVALID_ARG, "q or out is null or not 16-byte aligned");
  if (cfg->batch > 65535) return fail(HE_ERR_UNSUPPORTED, "batch %d > 65535 in one call", cfg->batch);
  AttendArgs a{*cfg, *cache, q, out};
  const dim3 grid((unsigned)cfg->n_kv_heads, (unsigned)cfg->batch);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int G = cfg->group_size, d = cfg->head_dim;
  if (cfg->dtype == HE_DTYPE_BF16 && d == 128 && getenv("HE_DISABLE_ATTEND_MMA") == nullptr) {
    // Cluster size: the largest power of two (<= 8) that keeps the grid within one CTA per SM.
    const long long units = (long long)cfg->batch * cfg->n_kv_heads;
    int sms = 0;
    if (int rc = sm_count(&sms)) return rc;
    int S = 1;
    while (S < 8 && units * (S * 2) <= sms) S *= 2;
    const size_t smem = (size_t)(kAttendWarps + 1) * G * (d + 2) * sizeof(float);
    if (int rc = set_smem(attend_bf16_kernel, smem)) return rc;
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3((unsigned)(cfg->n_kv_heads * S), (unsigned)cfg->batch);
    lc.blockDim = dim3(kAttendThreads);
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)S;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    lc.attrs = at;
    lc.numAttrs = 1;
    HE_CUDA_CHECK(cudaLaunchKernelEx(&lc, attend_bf16_kernel, a, S));
  } else {
    const size_t smem = ((size_t)G * d + (size_t)kAttendWarps * G * (d + 2)) * sizeof(float);
    if (int rc = set_smem(attend_generic_kernel, smem)) return rc;
    attend_generic_kernel<<<grid, kAttendThreads, smem, st>>>(a);
  }
  HE_CUDA_CHECK(cudaGetLastError());
  return HE_OK;
}

int he_decode_step_l2(const he_config* cfg, const he_cache* cache, const void* k, const void* v, int32_t* victim_out,
                      int32_t* evicted_pos_out, void* stream) {
  if (int rc = check_config(cfg, true)) return rc;
  if (int rc = check_cache(cache)) return rc;
  if (!k || !v || !victim_out) return fail(HE_ERR_INVALID_ARG, "k, v or victim_out is null");
  if (!aligned16(k) || !aligned16(v)) return fail(HE_ERR_INVALID_ARG, "k, v must be 16-byte aligned");
  if (cfg->batch > 65535) return fail(HE_ERR_UNSUPPORTED, "batch %d > 65535 in one decode call", cfg->batch);
  if (cfg->max_budget > 0xFFFFFF) return fail(HE_ERR_UNSUPPORTED, "max_budget %d too large", cfg->max_budget);
  StepL2Args a{*cfg, *cache, k, v, victim_out, evicted_pos_out};
  decode_step_l2_kernel<<<dim3((unsigned)cfg->n_kv_heads, (unsigned)cfg->batch), kStepL2Threads, 0, static_cast<cudaStream_t>(stream)>>>(a);
  HE_CUDA_CHECK(cudaGetLastError());
  return HE_OK;
}

int he_attention_loss(const he_config* cfg, const he_cache* cache, const void* q, const void* k_full,
                      const int64_t kv_strides[3], int32_t max_tokens, float* out, void* stream) {
  if (int rc = check_config(cfg, true)) return rc;
  if (int rc = check_cache(cache)) return rc;
  if (!q || !k_full || !kv_strides || !out) return fail(HE_ERR_INVALID_ARG, "q, k_full, kv_strides or out is null");
  if (!aligned16(q) || !aligned16(k_full)) return fail(HE_ERR_INVALID_ARG, "q and k_full must be 16-byte aligned");
  if (max_tokens < 0) return fail(HE_ERR_INVALID_ARG, "max_tokens %d < 0", max_tokens);
  const int es = esize_of(cfg->dtype);
  for (int i = 0; i < 3; ++i)
    if ((kv_strides[i] * es) % 16 != 0) return fail(HE_ERR_INVALID_ARG, "strides must keep every row 16-byte aligned");
  if (cfg->batch > 65535) return fail(HE_ERR_UNSUPPORTED, "batch %d > 65535 in one call", cfg->batch);
  const int G = cfg->group_size, d = cfg->head_dim;
  const bool fast = cfg->dtype == HE_DTYPE_BF16 && d == 128 && getenv("HE_DISABLE_ATTEND_MMA") == nullptr;
  const size_t smem = ((fast ? 0 : (size_t)G * d) + (size_t)kAttendWarps * G * 3) * sizeof(float) + ((size_t)max_tokens + 31) / 32 * 4 + 16;
  if (smem > 200 * 1024) return fail(HE_ERR_UNSUPPORTED, "max_tokens %d does not fit the kernel's bitmap", max_tokens);
  LossArgs a{*cfg, *cache, q, k_full, kv_strides[0], kv_strides[1], kv_strides[2], out};
  const dim3 grid((unsigned)cfg->n_kv_heads, (unsigned)cfg->batch);
  if (fast) {
    if (int rc = set_smem(attention_loss_bf16_kernel, smem)) return rc;
    attention_loss_bf16_kernel<<<grid, kAttendThreads, smem, static_cast<cudaStream_t>(stream)>>>(a);
  } else {
    if (int rc = set_smem(attention_loss_kernel, smem)) return rc;
    attention_loss_kernel<<<grid, kAttendThreads, smem, static_cast<cudaStream_t>(stream)>>>(a);
  }
  HE_CUDA_CHECK(cudaGetLastError());
  return HE_OK;
}

int he_reset(const he_config* cfg, const he_cache* cache, void* stream) {
  if (int rc = check_config(cfg, true)) return rc;
  if (int rc = check_cache(cache)) return rc;
  const long long slots = (long long)cfg->batch * cfg->n_kv_heads * cfg->max_budget;
  const int blocks = (int)((slots + 255) / 256 < 148 * 8 ? (slots + 255) / 256 : 148 * 8);
  reset_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(*cfg, *cache);
  HE_CUDA_CHECK(cudaGetLastError());
  return HE_OK;
}

size_t he_step_scratch_bytes(const he_config* cfg) {
  if (check_config(cfg, true) != HE_OK) return 0;
  return align_up((size_t)cfg->batch * cfg->n_kv_heads * (cfg->group_size + 1) * words_of(cfg->hash_bits) * 4, 256) +
         align_up(kWImageBytes, 256);
}

size_t he_decode_staging_bytes(const he_config* cfg) {
  if (check_config(cfg, true) != HE_OK) return 0;
  const size_t units = (size_t)cfg->batch * cfg->n_kv_heads;
  const size_t row = (size_t)cfg->head_dim * esize_of(cfg->dtype);
  return align_up(units * cfg->group_size * row, 256) + 2 * align_up(units * row, 256) + align_up(units * 4, 256);
}

int he_decode_step_host(const he_config* cfg, const he_cache* cache, const void* q_host, const void* k_host,
                        const void* v_host, int32_t* victim_host, void* staging, size_t staging_bytes, void* stream) {
  if (int rc = he_decode_step_host_enqueue(cfg, cache, q_host, k_host, v_host, victim_host, staging, staging_bytes, stream)) return rc;
  HE_CUDA_CHECK(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  return HE_OK;
}

int he_decode_step_host_enqueue(const he_config* cfg, const he_cache* cache, const void* q_host, const void* k_host,
                                const void* v_host, int32_t* victim_host, void* staging, size_t staging_bytes, void* stream) {
  if (int rc = check_config(cfg, true)) return rc;
  const bool block = q_host != nullptr && k_host == nullptr && v_host == nullptr;  // the one-block form (internal)
  if (!q_host || (!block && (!k_host || !v_host)) || !victim_host || !staging) return fail(HE_ERR_INVALID_ARG, "a host pointer or staging is null");
  if ((reinterpret_cast<uintptr_t>(staging) & 255u) != 0) return fail(HE_ERR_INVALID_ARG, "staging must be 256-byte aligned");
  const size_t need = he_decode_staging_bytes(cfg);
  if (staging_bytes < need) return fail(HE_ERR_WORKSPACE, "staging has %zu bytes, %zu needed", staging_bytes, need);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t units = (size_t)cfg->batch * cfg->n_kv_heads;
  const size_t row = (size_t)cfg->head_dim * esize_of(cfg->dtype);
  char* p = static_cast<char*>(staging);
  void* dq = p;
  p += align_up(units * cfg->group_size * row, 256);
  void* dk = p;
  p += align_up(units * row, 256);
  void* dv = p;
  p += align_up(units * row, 256);
  int32_t* dvictim = reinterpret_cast<int32_t*>(p);
  const size_t qb = units * cfg->group_size * row, kb = units * row;
  if (k_host == nullptr && v_host == nullptr) {
    // he_decode_step_host_block_enqueue: q, k, v in one host block laid out like the staging area, one copy. Every
    // driver call costs the host a few microseconds, and at these sizes (under 1 MB per step) that, not the bus, is
    // what an end-to-end step pays for first.
    HE_CUDA_CHECK(cudaMemcpyAsync(dq, q_host, align_up(qb, 256) + align_up(kb, 256) + kb, cudaMemcpyHostToDevice, st));
  } else {
    HE_CUDA_CHECK(cudaMemcpyAsync(dq, q_host, qb, cudaMemcpyHostToDevice, st));
    HE_CUDA_CHECK(cudaMemcpyAsync(dk, k_host, kb, cudaMemcpyHostToDevice, st));
    HE_CUDA_CHECK(cudaMemcpyAsync(dv, v_host, kb, cudaMemcpyHostToDevice, st));
  }
  if (int rc = he_decode_step(cfg, cache, dq, dk, dv, dvictim, nullptr, nullptr, stream)) return rc;
  HE_CUDA_CHECK(cudaMemcpyAsync(victim_host, dvictim, units * 4, cudaMemcpyDeviceToHost, st));
  return HE_OK;
}

size_t he_decode_host_block_bytes(const he_config* cfg, size_t offsets[3]) {
  if (check_config(cfg, true) != HE_OK) return 0;
  const size_t units = (size_t)cfg->batch * cfg->n_kv_heads;
  const size_t row = (size_t)cfg->head_dim * esize_of(cfg->dtype);
  const size_t qb = units * cfg->group_size * row, kb = units * row;
  if (offsets != nullptr) offsets[0] = 0, offsets[1] = align_up(qb, 256), offsets[2] = align_up(qb, 256) + align_up(kb, 256);
  return align_up(qb, 256) + align_up(kb, 256) + kb;
}

int he_decode_step_host_block_enqueue(const he_config* cfg, const he_cache* cache, const void* qkv_host, int32_t* victim_host,
                                      void* staging, size_t staging_bytes, void* stream) {
  if (qkv_host == nullptr) return fail(HE_ERR_INVALID_ARG, "qkv_host is null");
  return he_decode_step_host_enqueue(cfg, cache, qkv_host, nullptr, nullptr, victim_host, staging, staging_bytes, stream);
}

size_t he_prefill_staging_bytes(const he_config* cfg, int32_t max_prompt_len) {
  const size_t ws = he_workspace_bytes(cfg, max_prompt_len);
  if (ws == 0) return 0;
  const size_t units = (size_t)cfg->batch * cfg->n_kv_heads;
  const size_t rows = units * (size_t)max_prompt_len * cfg->head_dim * esize_of(cfg->dtype);
  return align_up(ws, 256) + align_up(rows * cfg->group_size, 256) + 2 * align_up(rows, 256) + align_up((size_t)cfg->batch * 4, 256);
}

int he_prefill_compress_host(const he_config* cfg, const he_cache* cache, const void* q_host, const void* k_host,
                             const void* v_host, const int32_t* prompt_len_host, int32_t max_prompt_len,
                             int32_t* fill_host, void* staging, size_t staging_bytes, void* stream) {
  if (int rc = check_config(cfg, true)) return rc;
  if (int rc = check_cache(cache)) return rc;
  if (!q_host || !k_host || !v_host || !prompt_len_host || !fill_host || !staging) return fail(HE_ERR_INVALID_ARG, "a host pointer or staging is null");
  if ((reinterpret_cast<uintptr_t>(staging) & 255u) != 0) return fail(HE_ERR_INVALID_ARG, "staging must be 256-byte aligned");
  if (max_prompt_len < 0) return fail(HE_ERR_INVALID_ARG, "max_prompt_len %d < 0", max_prompt_len);
  const size_t need = he_prefill_staging_bytes(cfg, max_prompt_len);
  if (staging_bytes < need) return fail(HE_ERR_WORKSPACE, "staging has %zu bytes, %zu needed", staging_bytes, need);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t units = (size_t)cfg->batch * cfg->n_kv_heads;
  const size_t rows = units * (size_t)max_prompt_len * cfg->head_dim * esize_of(cfg->dtype);
  const size_t ws = he_workspace_bytes(cfg, max_prompt_len);
  char* p = static_cast<char*>(staging);
  void* dws = p;
  p += align_up(ws, 256);
  void* dq = p;
  p += align_up(rows * cfg->group_size, 256);
  void* dk = p;
  p += align_up(rows, 256);
  void* dv = p;
  p += align_up(rows, 256);
  int32_t* dlen = reinterpret_cast<int32_t*>(p);
  HE_CUDA_CHECK(cudaMemcpyAsync(dq, q_host, rows * cfg->group_size, cudaMemcpyHostToDevice, st));
  HE_CUDA_CHECK(cudaMemcpyAsync(dk, k_host, rows, cudaMemcpyHostToDevice, st));
  HE_CUDA_CHECK(cudaMemcpyAsync(dv, v_host, rows, cudaMemcpyHostToDevice, st));
  HE_CUDA_CHECK(cudaMemcpyAsync(dlen, prompt_len_host, (size_t)cfg->batch * 4, cudaMemcpyHostToDevice, st));
  const int64_t N = max_prompt_len, d = cfg->head_dim;
  const int64_t qs[3] = {(int64_t)cfg->n_kv_heads * cfg->group_size * N * d, N * d, d};
  const int64_t ks[3] = {(int64_t)cfg->n_kv_heads * N * d, N * d, d};
  if (int rc = he_prefill_compress(cfg, cache, dq, dk, dv, qs, ks, dlen, max_prompt_len, dws, ws, stream)) return rc;
  HE_CUDA_CHECK(cudaMemcpyAsync(fill_host, cache->fill, units * 4, cudaMemcpyDeviceToHost, st));
  HE_CUDA_CHECK(cudaStreamSynchronize(st));
  return HE_OK;
}

}  // extern "C"
