/*
 * Seeded synthetic input generator for the HashEvict eviction path.
 *
 * This file is test/bench fixture code. It produces the K / Q / V / W tensors
 * that stand in for post-RoPE Llama activations. It contains none of the
 * method's arithmetic (no hashing, no Hamming distance, no eviction): both the
 * CPU oracle and the CUDA library only ever see the bytes written here.
 *
 * Every element is a pure function of (seed, stream, element index), so any
 * sub-block of a tensor can be produced on its own, in any order, on any
 * number of threads:
 *
 *   key(seed, stream)      = mix64(mix64(seed) ^ mix64(stream + GOLD))
 *   draw(key, i)           = mix64(key ^ mix64(i))                (splitmix64 finaliser)
 *   unit(u64)              = ((u64 >> 11) + 0.5) * 2^-53          in (0,1)
 *   normal(key, e)         : Box-Muller in double on pair p = e >> 1,
 *                            u1 = unit(draw(key,2p)), u2 = unit(draw(key,2p+1)),
 *                            r = sqrt(-2 ln u1); even e -> r cos(2 pi u2), odd e -> r sin(2 pi u2)
 *
 * Values are rounded once to the storage type (fp32, or bf16 round-to-nearest-even).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define HE_GEN_MAX_OUTLIERS 16
#define HE_GEN_MAX_CLUSTERS 64

typedef struct he_gen_spec {
  uint64_t seed;
  int32_t kind;          /* 0: iid N(0,1); 1: outlier channels + linear mean drift; 2: Gaussian clusters + outlier channels */
  int32_t dtype;         /* 0: fp32, 1: bf16 */
  int64_t n_heads;       /* heads per sequence in the index space */
  int64_t tok_space;     /* size of the token axis in the index space (prompt + decode tokens) */
  int64_t d;             /* channels */
  int32_t noise_stream;  /* stream id of the N(0,1) noise of this tensor */
  int32_t n_outlier;     /* kinds 1,2: outlier channels per (sequence, head) */
  double outlier_scale;  /* kinds 1,2: scale of an outlier channel */
  double drift_den;      /* kind 1: mean drift is m_c * token / drift_den */
  int32_t n_clusters;    /* kind 2 */
  int32_t pad_;
  double centre_scale;   /* kind 2: centres are centre_scale * N(0, I) */
  double sigma;          /* kind 2: within-cluster standard deviation */
} he_gen_spec;

enum { STREAM_OUTLIER = 7, STREAM_DRIFT = 8, STREAM_CENTRE = 9, STREAM_ASSIGN = 10 };

static inline uint64_t mix64(uint64_t z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
static inline uint64_t stream_key(uint64_t seed, uint64_t stream) {
  return mix64(mix64(seed) ^ mix64(stream + 0x9E3779B97F4A7C15ull));
}
static inline uint64_t draw(uint64_t key, uint64_t i) { return mix64(key ^ mix64(i)); }
static inline double unit01(uint64_t u) { return ((double)(u >> 11) + 0.5) * (1.0 / 9007199254740992.0); }

static inline double normal_at(uint64_t key, uint64_t e) {
  const uint64_t p = e >> 1;
  const double u1 = unit01(draw(key, 2 * p));
  const double u2 = unit01(draw(key, 2 * p + 1));
  const double r = sqrt(-2.0 * log(u1));
  const double th = 6.283185307179586476925286766559 * u2;
  return (e & 1) ? r * sin(th) : r * cos(th);
}

static inline uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7F800000u) == 0x7F800000u) return (uint16_t)(u >> 16); /* inf / nan: truncate */
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

/* Raw 64-bit draws: out[i] = draw(key(seed, stream), idx0 + i). */
void he_gen_u64(uint64_t seed, int32_t stream, uint64_t idx0, int64_t n, uint64_t* out) {
  const uint64_t key = stream_key(seed, (uint64_t)stream);
  for (int64_t i = 0; i < n; ++i) out[i] = draw(key, idx0 + (uint64_t)i);
}

/* Flat iid N(0,1) vector (used for W): out[i] = normal(key(seed,stream), idx0 + i) as fp32. */
void he_gen_normal_f32(uint64_t seed, int32_t stream, uint64_t idx0, int64_t n, float* out) {
  const uint64_t key = stream_key(seed, (uint64_t)stream);
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) out[i] = (float)normal_at(key, idx0 + (uint64_t)i);
}

static void outlier_channels(const he_gen_spec* s, uint64_t unit, int32_t* ch) {
  const uint64_t key = stream_key(s->seed, STREAM_OUTLIER);
  int found = 0;
  for (uint64_t attempt = 0; found < s->n_outlier && attempt < 4096; ++attempt) {
    const int32_t c = (int32_t)(draw(key, unit * 4096 + attempt) % (uint64_t)s->d);
    int dup = 0;
    for (int j = 0; j < found; ++j) dup |= (ch[j] == c);
    if (!dup) ch[found++] = c;
  }
}

/*
 * Fill the block [seq0, seq0+nseq) x all heads x tokens [tok0, tok0+ntok) x d of one tensor.
 * Element index (for the noise stream) = ((seq*n_heads + head)*tok_space + token)*d + c.
 * `out` points at element (seq0, head 0, tok0, 0); strides are in elements.
 */
void he_gen_fill(const he_gen_spec* s, int64_t seq0, int64_t nseq, int64_t tok0, int64_t ntok, void* out,
                 int64_t stride_seq, int64_t stride_head, int64_t stride_tok) {
  const uint64_t knoise = stream_key(s->seed, (uint64_t)s->noise_stream);
  const uint64_t kdrift = stream_key(s->seed, STREAM_DRIFT);
  const uint64_t kcentre = stream_key(s->seed, STREAM_CENTRE);
  const uint64_t kassign = stream_key(s->seed, STREAM_ASSIGN);
  const int64_t d = s->d;
  const int64_t nunits = nseq * s->n_heads;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t uu = 0; uu < nunits; ++uu) {
    const int64_t seq = seq0 + uu / s->n_heads;
    const int64_t head = uu % s->n_heads;
    const uint64_t unit = (uint64_t)(seq * s->n_heads + head);
    double* scale = (double*)malloc(sizeof(double) * (size_t)d * (2 + (s->kind == 2 ? (size_t)s->n_clusters : 0)));
    double* drift = scale + d;
    double* centres = drift + d; /* [n_clusters][d], kind 2 only */
    for (int64_t c = 0; c < d; ++c) { scale[c] = 1.0; drift[c] = 0.0; }
    if (s->kind == 1 || s->kind == 2) {
      int32_t ch[HE_GEN_MAX_OUTLIERS];
      outlier_channels(s, unit, ch);
      for (int j = 0; j < s->n_outlier; ++j) scale[ch[j]] = s->outlier_scale;
    }
    if (s->kind == 1)
      for (int64_t c = 0; c < d; ++c) drift[c] = normal_at(kdrift, unit * (uint64_t)d + (uint64_t)c) / s->drift_den;
    if (s->kind == 2)
      for (int64_t k = 0; k < s->n_clusters; ++k)
        for (int64_t c = 0; c < d; ++c)
          centres[k * d + c] =
              s->centre_scale * normal_at(kcentre, (unit * (uint64_t)s->n_clusters + (uint64_t)k) * (uint64_t)d + (uint64_t)c);
    char* base = (char*)out + ((seq - seq0) * stride_seq + head * stride_head) * (s->dtype ? 2 : 4);
    for (int64_t t = tok0; t < tok0 + ntok; ++t) {
      const uint64_t e0 = (unit * (uint64_t)s->tok_space + (uint64_t)t) * (uint64_t)d;
      const double* centre = centres;
      if (s->kind == 2)
        centre = centres + (int64_t)(draw(kassign, unit * (uint64_t)s->tok_space + (uint64_t)t) % (uint64_t)s->n_clusters) * d;
      char* row = base + (t - tok0) * stride_tok * (s->dtype ? 2 : 4);
      double z_odd = 0.0;
      for (int64_t c = 0; c < d; ++c) {
        /* e0 is even when d is even, so (c, c+1) is one Box-Muller pair; odd d falls back to per-element draws */
        double z;
        if ((d & 1) == 0) {
          if ((c & 1) == 0) {
            const uint64_t p = (e0 + (uint64_t)c) >> 1;
            const double u1 = unit01(draw(knoise, 2 * p));
            const double u2 = unit01(draw(knoise, 2 * p + 1));
            const double r = sqrt(-2.0 * log(u1));
            const double th = 6.283185307179586476925286766559 * u2;
            z = r * cos(th);
            z_odd = r * sin(th);
          } else {
            z = z_odd;
          }
        } else {
          z = normal_at(knoise, e0 + (uint64_t)c);
        }
        double val;
        if (s->kind == 0) val = z;
        else if (s->kind == 1) val = scale[c] * z + drift[c] * (double)t;
        else val = scale[c] * (centre[c] + s->sigma * z);
        if (s->dtype) ((uint16_t*)row)[c] = f32_to_bf16_rne((float)val);
        else ((float*)row)[c] = (float)val;
      }
    }
    free(scale);
  }
}
