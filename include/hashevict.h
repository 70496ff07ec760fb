/*
 * hashevict.h - C ABI of the HashEvict eviction hot path for NVIDIA B200 (sm_100a).
 *
 * The library keeps, per (sequence, KV head) "unit", a key/value cache of at most C slots and a
 * table of b-bit SimHash codes of the cached keys. Each decode step hashes the new query and key,
 * scores every cached key by Hamming distance to the query code, and overwrites the slot with
 * the lowest score by the new token (Section 3: Eq. 4-6 and Algorithm 1). The prefill call does
 * the same for a whole prompt (Section 3, "Prompt Encoding Stage").
 *
 * General rules for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller unless a parameter says "host".
 *     The library allocates no memory; scratch space is passed in by the caller (the one exception,
 *     he_prefill_compress_noalloc, uses an array that is part of the library's device image).
 *   - Calls only enqueue work on `stream` (a cudaStream_t passed as void*) and return at once;
 *     they never synchronise (the *_host variants are the exception and say so). Results are
 *     valid once the stream has been synchronised.
 *   - The return value is a status code (HE_OK = 0). No exception crosses this boundary.
 *     he_last_error() returns a human-readable description of the calling thread's last failure.
 *   - There is no CPU fallback: without a CUDA device every compute call fails with HE_ERR_CUDA.
 *
 * Layouts (B sequences, Hkv KV heads, G query heads per KV head, d = head_dim, b = hash_bits,
 * Wd = ceil(b/32), Cmax = max_budget = slot stride, unit u = s*Hkv + h):
 *   k_cache, v_cache  [B, Hkv, Cmax, d]   dtype of the config, rows 16-byte aligned
 *   codes             [B, Hkv, Cmax, Wd]  uint32; bit i of a code is the sign bit of column i of W,
 *                                         stored in word i/32 at bit i%32; unused high bits are 0
 *                                         With HE_FLAG_PACKED_CODES: [B, Hkv, Cmax, ceil(b/8)] bytes instead, bit i in
 *                                         byte i/8 at bit i%8 (1 byte per slot at b <= 8, as Section 4.7 prices it);
 *                                         Cmax * ceil(b/8) must then be a multiple of 16. For b = 32 and b = 64 the
 *                                         two layouts are the same bytes.
 *   scores            [B, Hkv, Cmax]      fp32, -(Hamming distance summed over the group)
 *   pos               [B, Hkv, Cmax]      int32 token position held by the slot, -1 = empty
 *   budget            [B]                 int32, 1 <= C_s <= Cmax, read-only. Checked on the host only when
 *                                         he_cache.budget_host is given (HE_ERR_INVALID_ARG); on the device a value
 *                                         above Cmax counts as Cmax and a value below 1 as "this sequence stores
 *                                         nothing" (prefill leaves its units empty, decode leaves them untouched and
 *                                         reports victim -1).
 *   fill, next_pos    [B, Hkv]            int32 valid slots / position of the next token, per unit
 *   W                 [d, b]              fp32 row-major: W = R^T of Eq. 2, read-only while in use
 */
#ifndef HASHEVICT_H_
#define HASHEVICT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  HE_OK = 0,
  HE_ERR_INVALID_ARG = 1, /* null or misaligned pointer, size out of range */
  HE_ERR_UNSUPPORTED = 2, /* shape outside what the kernels were built for */
  HE_ERR_CUDA = 3,        /* a CUDA runtime call or launch failed */
  HE_ERR_WORKSPACE = 4    /* caller-provided scratch too small */
};

enum { HE_DTYPE_F32 = 0, HE_DTYPE_BF16 = 1 };

/* flags */
#define HE_FLAG_WRITE_SCORES 1u /* store the per-slot scores of Eq. 5 on every evicting step */
#define HE_FLAG_PACKED_CODES 2u /* he_cache.codes holds ceil(b/8) bytes per slot instead of Wd 32-bit words */
#define HE_FLAG_EARLY_INPUTS 4u /* he_decode_step may read q, k, v before the stream's earlier work has finished:
                                   see he_decode_step */

typedef struct he_config {
  int32_t batch;      /* B; independent layers may be folded in by the caller */
  int32_t n_kv_heads; /* Hkv */
  int32_t group_size; /* G >= 1; the G query heads of a KV head add their Hamming distances */
  int32_t head_dim;   /* d, a multiple of 8, <= 256 */
  int32_t hash_bits;  /* b in [1, 64] */
  int32_t max_budget; /* Cmax: slot stride of the cache arrays, a multiple of 4, <= 2^20 */
  int32_t n_sink;     /* tokens at positions < n_sink are never evicted (0 = plain Algorithm 1) */
  int32_t n_recent;   /* the n_recent newest cached tokens are never evicted (0 = plain Algorithm 1) */
  int32_t dtype;      /* HE_DTYPE_* of q, k, v and of the K/V caches */
  uint32_t flags;     /* HE_FLAG_* */
} he_config;

typedef struct he_cache {
  void* k_cache;
  void* v_cache;
  uint32_t* codes;
  float* scores;
  int32_t* pos;
  const int32_t* budget;
  int32_t* fill;
  int32_t* next_pos;
  const float* W;
  const int32_t* budget_host; /* optional HOST copy of budget ([B]), or NULL. When given (and B <= 1024)
                                 he_decode_step passes the budgets in the kernel parameters, which saves the
                                 kernel one dependent device read before it can start streaming the code table.
                                 With protected windows (n_sink or n_recent > 0) he_prefill_compress also needs it to
                                 check that every budget exceeds n_sink + n_recent before it picks its faster replay
                                 kernel; without it the call is correct but slower. Must hold the same values as `budget`. */
  uint32_t* step_scratch;     /* optional device buffer of he_step_scratch_bytes(cfg) bytes, or NULL. When given and
                                 a step has at least 16384 new rows (B * Hkv * (G + 1)), he_decode_step first hashes
                                 all of them with the bulk projection kernels into this buffer and the per-unit
                                 kernel only scans; results are the same as with the single fused kernel. */
} he_cache;

/*
 * he_hash_keys - SimHash codes of `rows` vectors (keys or queries alike), Eq. 2:
 *   code bit i of row r = [ sum_c x[r, c] * W[c, i] >= 0 ]   (sgn(0) = 1).
 * x: [rows, d] with a row stride of `row_stride_elems` elements (>= d, rows 16-byte aligned),
 * dtype from cfg. codes_out: [rows, Wd] uint32. Only head_dim, hash_bits and dtype of cfg are used.
 * The projection is accumulated in fp32; a bit may differ from exact arithmetic only where the
 * exact projection is within 1e-5 * |x| * |W[:, i]| of zero. rows = 0 is a no-op.
 */
int he_hash_keys(const he_config* cfg, const void* x, int64_t rows, int64_t row_stride_elems, const float* W,
                 uint32_t* codes_out, void* stream);

/*
 * he_decode_step - one application of Algorithm 1, lines 1-5, to every unit ("Decoding Stage").
 * q: [B, Hkv*G, d], k, v: [B, Hkv, d] (contiguous). For each unit, with t = next_pos:
 *   cache not full (fill < C_s): the token is appended at slot fill; nothing is scored;
 *   otherwise D_j = sum_g popcount(codes[j] xor h(q_g)) for every slot (Eq. 5, score_j = -D_j),
 *   the victim is the lowest-index eligible slot with the largest D_j (Eq. 6); a slot is eligible
 *   when n_sink <= pos_j < t - n_recent (if no slot is eligible, all are).
 * Then K, V, code and pos of that slot are overwritten by k, v, h(k), t; next_pos and fill advance.
 * victim_out [B, Hkv]: slot written. evicted_pos_out [B, Hkv] (nullable): position that was evicted,
 * -1 when appended. qcodes_out [B, Hkv*G, Wd] (nullable): the query codes that were used.
 * The scores array is written only with HE_FLAG_WRITE_SCORES. A sequence whose budget is < 1 holds nothing: its units
 * are left untouched and report victim -1.
 *
 * Ordering against earlier work of the stream. The kernel is launched with the programmatic-serialization attribute,
 * so it may start while the stream's previous kernel is still running. By default it reads only W (which must not
 * change while the cache is in use) before it waits for that kernel to finish; q, k, v may therefore be produced by
 * the kernel enqueued just before this call. With HE_FLAG_EARLY_INPUTS the call also reads q, k, v and hashes them
 * (Eq. 2) BEFORE that wait, so that this work overlaps the previous call's scan: consecutive decode calls (say, the
 * caches of a model's layers one after another, or one cache step after step) then run about twice as fast. The
 * caller promises in exchange that q, k, v were completely written before this call was ENQUEUED on the stream's
 * device timeline - by work the host has synchronised with, or by work ordered before everything still pending in
 * the stream (inputs staged ahead of a run of calls, or a captured graph whose inputs are final before it is
 * launched). If the rows are produced by a kernel enqueued shortly before the call, leave the flag off. Results are
 * identical with and without the flag.
 */
int he_decode_step(const he_config* cfg, const he_cache* cache, const void* q, const void* k, const void* v,
                   int32_t* victim_out, int32_t* evicted_pos_out, uint32_t* qcodes_out, void* stream);

/*
 * he_prefill_compress - "Prompt Encoding Stage": the cache is reset, the first C_s prompt tokens fill
 * slots 0..C_s-1, and every later prompt token t = C_s..N_s-1 goes through Algorithm 1 in order, so
 * the result equals he_reset followed by N_s calls of he_decode_step - given the same hash bits. The bulk
 * projection of the prompt (tensor cores for bf16 rows) and the projection inside a decode step round the same sum
 * differently, so a bit whose exact projection lies within 1e-5 * |x| * |w| of zero (about one in 1e4 to 1e5 bits)
 * may come out differently on the two routes, and the two caches then part ways from that token on; each route on
 * its own is a valid run of Algorithm 1 under Eq. 2's tolerance.
 * q: [B, Hkv*G, N, d], k, v: [B, Hkv, N, d] addressed with element strides (batch, head, token);
 * channels are contiguous and every row is 16-byte aligned. prompt_len: [B] int32 on the device,
 * each <= max_prompt_len (a larger value counts as max_prompt_len, a negative one as 0). Queries of tokens that
 * are appended are never read.
 * workspace: at least he_workspace_bytes(cfg, max_prompt_len) bytes, 256-byte aligned; it receives
 * the prompt codes: key codes [B*Hkv, Nmax, Wd] followed by query codes [B*Hkv, Nmax, G, Wd]
 * (query codes of appended tokens are left unwritten). scores hold the last evicting step's values.
 */
int he_prefill_compress(const he_config* cfg, const he_cache* cache, const void* q, const void* k, const void* v,
                        const int64_t q_strides[3], const int64_t kv_strides[3], const int32_t* prompt_len,
                        int32_t max_prompt_len, void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of he_cache.step_scratch: the codes of one decode step's new rows, (G + 1) * Wd words per unit, plus the
   three-term bf16 image of W that the bulk projection kernels read (0 on bad input). */
size_t he_step_scratch_bytes(const he_config* cfg);

/* Scratch bytes he_prefill_compress needs for prompts of up to max_prompt_len tokens (0 on bad input). */
size_t he_workspace_bytes(const he_config* cfg, int32_t max_prompt_len);

/*
 * he_attend - attention over the compressed cache, the step that follows the eviction (Algorithm 1 line 6, Eq. 1):
 *   out[s, h*G + g, :] = sum_j softmax_j( q[s, h*G + g, :] . K[s, h, j, :] / sqrt(d) ) * V[s, h, j, :]
 * over the valid slots j < fill of unit (s, h). q: [B, Hkv*G, d] in the dtype of cfg (contiguous); out: [B, Hkv*G, d]
 * fp32. Products of bf16 inputs are exact; sums and the softmax are carried in fp32 (exp2 of scaled scores, running
 * maximum), so results agree with exact arithmetic to about 1e-5 of the largest |V| entry. A unit without valid
 * slots gives zeros. The cache is only read.
 */
int he_attend(const he_config* cfg, const he_cache* cache, const void* q, float* out, void* stream);

/* he_reset - empty every unit: fill = 0, next_pos = 0, pos = -1, codes = 0, scores = 0. K/V are left as they are. */
int he_reset(const he_config* cfg, const he_cache* cache, void* stream);

/*
 * Host-buffer variants: the same calls for callers whose activations live in (preferably pinned)
 * HOST memory. They copy the inputs to `staging` on `stream`, run the device call, copy the result
 * back and synchronise `stream` before returning.
 *   he_decode_step_host:  q/k/v are host pointers laid out as for he_decode_step; victim_host [B, Hkv]
 *     receives the slots written. staging: >= he_decode_staging_bytes(cfg) device bytes.
 *   he_decode_step_host_enqueue: the same copies and kernels put on `stream` WITHOUT the final synchronise, so that a
 *     caller can keep several streams busy (say, the caches of different layers on alternating streams, each with
 *     its own staging, copies of one overlapping the kernel of the other). victim_host holds the result, and
 *     q/k/v_host and staging may be reused, only once `stream` has been synchronised; the host buffers must be
 *     pinned for the copies to be asynchronous.
 *   he_decode_step_host_block_enqueue: the same with q, k, v in ONE host block (one pinned allocation), q at offset 0,
 *     k and v at the offsets he_decode_host_block_bytes reports (each tensor starts on the next 256-byte boundary; the
 *     function returns the block's size). The block travels in a single copy: three driver calls per step instead of
 *     five, which matters because at under 1 MB per step the calls cost the host more than the bus costs the copy.
 *   he_prefill_compress_host: q [B, Hkv*G, Nmax, d], k, v [B, Hkv, Nmax, d] contiguous host tensors,
 *     prompt_len_host [B]; fill_host [B, Hkv] receives the valid-slot counts. staging: >=
 *     he_prefill_staging_bytes(cfg, max_prompt_len) device bytes (includes the prompt-code workspace).
 */
size_t he_decode_staging_bytes(const he_config* cfg);
int he_decode_step_host(const he_config* cfg, const he_cache* cache, const void* q_host, const void* k_host,
                        const void* v_host, int32_t* victim_host, void* staging, size_t staging_bytes, void* stream);
int he_decode_step_host_enqueue(const he_config* cfg, const he_cache* cache, const void* q_host, const void* k_host,
                                const void* v_host, int32_t* victim_host, void* staging, size_t staging_bytes, void* stream);
size_t he_decode_host_block_bytes(const he_config* cfg, size_t offsets[3]);
int he_decode_step_host_block_enqueue(const he_config* cfg, const he_cache* cache, const void* qkv_host, int32_t* victim_host,
                                      void* staging, size_t staging_bytes, void* stream);
size_t he_prefill_staging_bytes(const he_config* cfg, int32_t max_prompt_len);
int he_prefill_compress_host(const he_config* cfg, const he_cache* cache, const void* q_host, const void* k_host,
                             const void* v_host, const int32_t* prompt_len_host, int32_t max_prompt_len,
                             int32_t* fill_host, void* staging, size_t staging_bytes, void* stream);

/*
 * he_prefill_oneshot - prompt compression by the one-shot ranking of Appendix C instead of Algorithm 1: for every
 * prompt token i the Hamming distance of its key code to the query codes of all later tokens j > i (summed over the
 * group's G query heads as in Eq. 5) is averaged over those tokens, and the min(N, C) tokens with the lowest average
 * stay. The paper uses this ranking only to analyse the method; it is NOT the procedure of Section 3 and gives a
 * different cache. Order: tokens inside the protected windows (i < n_sink or i >= N - n_recent) first, in token
 * order; then by average, compared exactly as fractions; equal averages by token index; the prompt's last token has
 * no later query and counts as average 0. Kept tokens are stored in token order: slot s holds the s-th kept token
 * (K, V, code, position; score = -(float)S / (float)n with S the summed distance and n = N - 1 - i, 0 when n = 0);
 * fill = min(N, C), next_pos = N, everything beyond fill is reset. Arguments, layouts, strides and errors are those
 * of he_prefill_compress, except: workspace >= he_oneshot_workspace_bytes(cfg, max_prompt_len) bytes;
 * max_prompt_len <= 32768; sums_out (device, nullable) [B, Hkv, max_prompt_len] int64 receives S for every prompt
 * token (entries beyond a sequence's length are not written). All arithmetic is integer except the stored score.
 */
size_t he_oneshot_workspace_bytes(const he_config* cfg, int32_t max_prompt_len);
int he_prefill_oneshot(const he_config* cfg, const he_cache* cache, const void* q, const void* k, const void* v,
                       const int64_t q_strides[3], const int64_t kv_strides[3], const int32_t* prompt_len,
                       int32_t max_prompt_len, void* workspace, size_t workspace_bytes, long long* sums_out, void* stream);

/*
 * he_prefill_oneshot_l2 - the comparison policy the paper names (Section 1, Section 4 setup: dropping tokens by the
 * high L2 norm of their key embeddings; Appendix B: "a low-to-high ordering of all L2 key norms") as a one-shot prompt
 * compression under the same boundary. Not HashEvict: it is here so that both policies can be measured on the same
 * cache layout. Order: protected tokens first (token order), then by squared key norm ascending, equal norms by
 * token index; the first min(N, C) stay, stored in token order. The norm is taken in fp32 with channels in ascending
 * order, one fused multiply-add per channel starting from 0 (this precision decides the ranking). Slot s holds the
 * s-th kept token: K, V, its Eq. 2 code (the cache stays a valid state for he_decode_step), position, score = -norm2.
 * No queries are read. workspace >= he_oneshot_workspace_bytes(cfg, max_prompt_len); max_prompt_len <= 32768;
 * norms_out (device, nullable) [B, Hkv, max_prompt_len] fp32 receives norm2 of every prompt key.
 */
int he_prefill_oneshot_l2(const he_config* cfg, const he_cache* cache, const void* k, const void* v, const int64_t kv_strides[3],
                          const int32_t* prompt_len, int32_t max_prompt_len, void* workspace, size_t workspace_bytes,
                          float* norms_out, void* stream);

/*
 * he_decode_step_l2 - one decoding step of the same comparison policy under the boundary of he_decode_step: the new
 * token always enters; while a unit's cache is full, the resident token with the highest squared key norm leaves
 * (lowest slot on equal norms; protected windows and the "if no slot is eligible, all are" rule as in
 * he_decode_step). It relies on scores[j] = -norm2 of the key in slot j, as he_prefill_oneshot_l2 and this call leave
 * them; mixing it with he_decode_step on one cache is not meaningful. The slot's code is set to zero. k, v:
 * [B, Hkv, d] contiguous device rows; victim_out [B, Hkv] (required), evicted_pos_out [B, Hkv] (nullable, -1 while
 * appending). No queries are read.
 */
int he_decode_step_l2(const he_config* cfg, const he_cache* cache, const void* k, const void* v, int32_t* victim_out,
                      int32_t* evicted_pos_out, void* stream);

/*
 * he_attention_loss - attention loss of the compressed cache (Section 4.6, Appendix B): for every unit and each of its
 * G query heads, out = sum of softmax_p(q . k_p / sqrt(d)) over the tokens p < next_pos that are NOT in the cache,
 * i.e. 1 - the attention mass of the cached tokens, the softmax being over ALL next_pos tokens seen so far.
 * q [B, Hkv*G, d] (cfg dtype, contiguous); k_full: every key seen so far, strided [B, Hkv, n, d] with element strides
 * kv_strides (batch, head, token), n >= next_pos of every unit and n <= max_tokens; out [B, Hkv*G] fp32. The dropped
 * mass is summed directly in fp32 (online maximum), so small losses keep their relative accuracy (about 1e-5). A unit
 * that has seen no token gives 0. The cache is only read.
 */
int he_attention_loss(const he_config* cfg, const he_cache* cache, const void* q, const void* k_full,
                      const int64_t kv_strides[3], int32_t max_tokens, float* out, void* stream);

/*
 * he_prefill_compress_noalloc - he_prefill_compress for callers that cannot obtain device memory for the
 * prompt-code workspace. (The paper has no counterpart: this is a packaging variant, the computation and the
 * results are those of he_prefill_compress.)
 *
 * Who needs it: code that runs where allocating is not possible or not allowed - inside a serving loop whose
 * memory pool is fully committed to the KV cache, in a plug-in that receives raw pointers but no allocator, or
 * in a process that must not call cudaMalloc once it has started (allocation synchronises the device and can
 * fail late). Such callers still pass their inputs and the cache arrays; only the scratch is provided here.
 *
 * The scratch is a fixed array of HE_NOALLOC_SCRATCH_BYTES bytes that lives in the library's device image:
 * every GPU that loads the library holds it until the process exits. The call fails with HE_ERR_WORKSPACE,
 * and does nothing, when he_workspace_bytes(cfg, max_prompt_len) exceeds that size. It never calls cudaMalloc,
 * cudaFree or any allocating routine.
 *
 * The first call on each device looks up the array's device address (one cudaGetSymbolAddress with that device
 * current); make that first call outside of any stream capture. All calls share the one array and it keeps
 * whatever the previous call wrote: nothing in it needs to start at zero, but two calls whose kernels overlap
 * on the GPU (different streams, no ordering between them) would overwrite each other's prompt codes - order
 * them on one stream or with events. After the call the prompt codes are in the array only until the next call.
 * All other arguments, layouts and error codes are those of he_prefill_compress.
 */
#define HE_NOALLOC_SCRATCH_BYTES (16u << 20)
int he_prefill_compress_noalloc(const he_config* cfg, const he_cache* cache, const void* q, const void* k,
                                const void* v, const int64_t q_strides[3], const int64_t kv_strides[3],
                                const int32_t* prompt_len, int32_t max_prompt_len, void* stream);

/*
 * he_device_error_count - how many thread blocks of this library's kernels gave up on a bounded device-side
 * wait since the library was loaded (0 in a healthy process; the kernels never wait without a limit, and a
 * block that hits one releases what it holds and returns), plus, in the bounds-checking debug build, how many
 * indices were found out of range. A call during which the counter rose has returned HE_OK all the same (calls
 * only enqueue work), but its outputs are undefined: he_hash_keys, he_prefill_compress and its variants, and
 * he_decode_step with a step scratch are the calls whose kernels contain such waits. This is the one call of the
 * library, besides the *_host variants, that synchronises the device. Returns -1 if the counter cannot be read.
 * Diagnostic only: the paper has no counterpart.
 */
int he_device_error_count(void);

/*
 * he_prefill_phase_events - timing aid (the paper has no counterpart). events: five cudaEvent_t handles (as void*)
 * created by the caller with timing enabled, or NULL to switch the aid off. While set, every prefill call of the
 * calling thread (he_prefill_compress and its variants) records them on its stream around its phases, launching
 * exactly the kernels it always launches: [0] start, [1] after Eq. 2 on the prompt keys (with the W image), [2] after
 * Eq. 2 on the queries, [3] after the unit schedule and the replay (or ranking), [4] after the K / V gather. An event
 * record is one more stream operation between two kernels, so use it for measurement runs only.
 */
int he_prefill_phase_events(void* const* events);

/* Text of the calling thread's most recent error ("" if none). The pointer stays valid until the next failing call. */
const char* he_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* HASHEVICT_H_ */
