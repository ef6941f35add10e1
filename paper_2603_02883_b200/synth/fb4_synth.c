/*
 * Seeded synthetic inputs for the FB4 quantizer: activation tensors, per-token
 * attention scores and SeDA cluster assignments.
 *
 * This file holds NO part of the quantization method.  It only produces input
 * data, and it is the one module that both the CPU oracle's tests and the CUDA
 * path's tests/benchmarks draw their inputs from.
 *
 * Every value is a pure function of (seed, stream, index): a counter-based
 * generator built from the splitmix64 finaliser, so any row of any tensor can be
 * produced on its own (the full-size parity tests sample rows) and the bytes do
 * not depend on thread count or on the PyTorch/numpy version.
 *
 * Activation recipes (they stand in for video-DiT linear-layer inputs, which are
 * heavy-tailed per token and carry a few large-magnitude outlier channels):
 *   kind 0: x[t][c] = z            z ~ N(0,1)
 *   kind 1: x[t][c] = s_t * tau    s_t = exp(N(0,1)) per token,
 *                                  tau ~ Student-t(nu=3) = z0 / sqrt((z1^2+z2^2+z3^2)/3)
 * then x[t][c] *= outlier_gain for c in a seeded set of distinct outlier channels,
 * and the result is rounded to bfloat16 (round-to-nearest-even).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define FB4S_PI 3.14159265358979323846

static inline uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xbf58476d1ce4e5b9ULL;
  z = (z ^ (z >> 27)) * 0x94d049bb133111ebULL;
  return z ^ (z >> 31);
}

/* 64 random bits for (seed, stream, counter). */
static inline uint64_t rnd64(uint64_t seed, uint64_t stream, uint64_t ctr) {
  uint64_t k = mix64(seed * 0x9e3779b97f4a7c15ULL + 0x632be59bd9b4e019ULL);
  k = mix64(k ^ (stream * 0xd1342543de82ef95ULL + 0x2545f4914f6cdd1dULL));
  return mix64(k + ctr * 0x9e3779b97f4a7c15ULL);
}

/* uniform in (0,1] with 53 bits */
static inline double u01_open0(uint64_t r) { return ((double)(r >> 11) + 1.0) * (1.0 / 9007199254740992.0); }
/* uniform in [0,1) with 53 bits */
static inline double u01(uint64_t r) { return (double)(r >> 11) * (1.0 / 9007199254740992.0); }

/* Two independent N(0,1) from counter pair (2*ctr, 2*ctr+1): Box-Muller. */
static inline void normal2(uint64_t seed, uint64_t stream, uint64_t ctr, double *z0, double *z1) {
  double u1 = u01_open0(rnd64(seed, stream, 2 * ctr));
  double u2 = u01(rnd64(seed, stream, 2 * ctr + 1));
  double r = sqrt(-2.0 * log(u1));
  double a = 2.0 * FB4S_PI * u2;
  *z0 = r * cos(a);
  *z1 = r * sin(a);
}

static inline uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7f800000u) == 0x7f800000u) return (uint16_t)(u >> 16); /* inf/nan: truncate */
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  return (uint16_t)(u >> 16);
}

enum { STREAM_DATA = 1, STREAM_TOKEN_SCALE = 2, STREAM_OUTLIER = 3, STREAM_SCORE = 4,
       STREAM_CUTS = 5, STREAM_SUBBOOK = 6 };

/*
 * Seeded set of n distinct channel indices in [0, C): partial Fisher-Yates over
 * an index array, driven by the counter generator.  out must hold n entries.
 */
int fb4s_outlier_channels(uint64_t seed, int64_t C, int64_t n, int64_t *out) {
  if (n < 0 || n > C || C <= 0) return -1;
  int64_t *perm = (int64_t *)malloc((size_t)C * sizeof(int64_t));
  if (!perm) return -2;
  for (int64_t i = 0; i < C; ++i) perm[i] = i;
  for (int64_t i = 0; i < n; ++i) {
    uint64_t r = rnd64(seed, STREAM_OUTLIER, (uint64_t)i);
    int64_t j = i + (int64_t)(r % (uint64_t)(C - i));
    int64_t tmp = perm[i]; perm[i] = perm[j]; perm[j] = tmp;
    out[i] = perm[i];
  }
  free(perm);
  return 0;
}

/*
 * Fill rows [row0, row0+nrows) of the T x C activation tensor (bf16 bit patterns,
 * row-major, `ld` elements between rows of `out`).  `gain[c]` is the per-channel
 * multiplier (1 or the outlier gain), supplied by the caller.
 */
int fb4s_fill_rows(uint64_t seed, int kind, int64_t C, int64_t row0, int64_t nrows,
                   const float *gain, uint16_t *out, int64_t ld) {
  if (C <= 0 || nrows < 0 || ld < C) return -1;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < nrows; ++r) {
    int64_t t = row0 + r;
    uint16_t *o = out + r * ld;
    if (kind == 0) {
      for (int64_t c = 0; c < C; c += 2) {
        double z0, z1;
        normal2(seed, STREAM_DATA, (uint64_t)(t * ((C + 1) / 2) + c / 2), &z0, &z1);
        o[c] = f32_to_bf16_rne((float)(z0 * gain[c]));
        if (c + 1 < C) o[c + 1] = f32_to_bf16_rne((float)(z1 * gain[c + 1]));
      }
    } else {
      double zs, zunused;
      normal2(seed, STREAM_TOKEN_SCALE, (uint64_t)t, &zs, &zunused);
      double s = exp(zs);
      for (int64_t c = 0; c < C; ++c) {
        double z0, z1, z2, z3;
        uint64_t e = (uint64_t)(t * C + c);
        normal2(seed, STREAM_DATA, 2 * e, &z0, &z1);
        normal2(seed, STREAM_DATA, 2 * e + 1, &z2, &z3);
        double tau = z0 / sqrt((z1 * z1 + z2 * z2 + z3 * z3) / 3.0);
        o[c] = f32_to_bf16_rne((float)(s * tau * gain[c]));
      }
    }
  }
  return 0;
}

/* Per-token attention scores, uniform in [0,1) as fp32. */
int fb4s_scores(uint64_t seed, int64_t t0, int64_t n, float *out) {
  for (int64_t i = 0; i < n; ++i) {
    /* 24 random bits so the fp32 value is exact and < 1 */
    out[i] = (float)(rnd64(seed, STREAM_SCORE, (uint64_t)(t0 + i)) >> 40) * (1.0f / 16777216.0f);
  }
  return 0;
}

static int cmp_i64(const void *a, const void *b) {
  int64_t x = *(const int64_t *)a, y = *(const int64_t *)b;
  return (x > y) - (x < y);
}

/*
 * n_clusters contiguous token ranges covering [0,T): n_clusters-1 distinct seeded
 * cut points in [1,T-1], sorted; cluster_id[t] = number of cuts <= t.
 */
int fb4s_cluster_ids(uint64_t seed, int64_t T, int32_t n_clusters, int32_t *cluster_id) {
  if (n_clusters < 1 || (int64_t)n_clusters > T) return -1;
  int64_t ncut = n_clusters - 1;
  int64_t *cuts = (int64_t *)malloc((size_t)(ncut + 1) * sizeof(int64_t));
  if (!cuts) return -2;
  /* distinct values by rejection (ncut << T in every use) */
  int64_t have = 0;
  uint64_t ctr = 0;
  while (have < ncut) {
    int64_t c = 1 + (int64_t)(rnd64(seed, STREAM_CUTS, ctr++) % (uint64_t)(T - 1));
    int dup = 0;
    for (int64_t i = 0; i < have; ++i) if (cuts[i] == c) { dup = 1; break; }
    if (!dup) cuts[have++] = c;
  }
  qsort(cuts, (size_t)ncut, sizeof(int64_t), cmp_i64);
  int64_t k = 0;
  for (int64_t t = 0; t < T; ++t) {
    while (k < ncut && cuts[k] <= t) ++k;
    cluster_id[t] = (int32_t)k;
  }
  free(cuts);
  return 0;
}

/*
 * One seeded 8-dialect sub-formatbook per cluster: for every dynamic-range bucket
 * (largest magnitude 8..15) pick one seeded member among the dialects of the
 * given 32x8 formatbook whose largest magnitude equals the bucket.  Buckets with
 * no dialect contribute nothing.  mask[k] bit d set <=> dialect d allowed.
 */
int fb4s_cluster_masks(uint64_t seed, const uint8_t *formatbook, int32_t n_clusters, uint32_t *mask) {
  for (int32_t k = 0; k < n_clusters; ++k) {
    uint32_t m = 0;
    for (int b = 8; b <= 15; ++b) {
      int members[32], n = 0;
      for (int d = 0; d < 32; ++d) if (formatbook[d * 8 + 7] == b) members[n++] = d;
      if (n == 0) continue;
      uint64_t r = rnd64(seed, STREAM_SUBBOOK, (uint64_t)k * 16 + (uint64_t)b);
      m |= 1u << members[r % (uint64_t)n];
    }
    mask[k] = m;
  }
  return 0;
}
