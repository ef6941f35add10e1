/*
 * fb4_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, table-free CPU statement of what the FB4 online activation
 * quantizer computes (SemanticDialect, Sec. 3.1-3.4), used only to check the
 * CUDA library and to time a CPU baseline.  Only the tests, the smoke check and
 * the benchmark's cpu-baseline/reference legs may call it; the CUDA library
 * never does, and the two share no code, headers, tables or constants.
 *
 * Everything is done by direct arithmetic in double precision / integers, one
 * block at a time, in the order the paper gives:
 *   Sec. 3.1  block normalisation: power-of-two scale from floor(log2(amax)),
 *             exponent offset by 3 so normalised magnitudes v lie in [0,16)
 *             with the block maximum in [8,16); 1 sign bit + 3-bit index into
 *             the block's dialect (8 integer magnitudes 0..15).
 *   Sec. 3.2  group-wise maxima (num_groups contiguous groups), approximate
 *             error of a dialect = sum over group maxima of the absolute error
 *             at the midpoint of the maximum's 0.5-wide bin; two-stage
 *             selection (sub-formatbook by block maximum, then argmin); every
 *             element then rounds to the nearest magnitude of the chosen dialect.
 *   Sec. 3.3  activation decomposition: residual Delta = Act - Q(Act) of the
 *             salient tokens is quantized again; one salient token per tile,
 *             the highest-scoring one.
 *   Sec. 3.3 / App. C  weights are quantized offline with exhaustive selection: the
 *             squared error of every dialect over all elements of the block, minimum wins.
 *   App. D.2  MXFP8 view: the integer magnitudes 0..15 are exact in FP8 e4m3 and the
 *             power-of-two block scale is an E8M0 scale, so a quantized tensor can be
 *             re-expressed as an MXFP8 operand without any rounding.
 *   App. D.2  fusion with the preceding operation: the per-channel affine step y = x * g_c +
 *             bias_c (LayerNorm tail / modulation) in float32 with one rounding, and the
 *             quantizer on float32 values taken as they are.
 *   Sec. 3.4  SeDA: the candidate set of a token is its cluster's sub-formatbook; a
 *             sub-formatbook is built by counting, over a cluster's anchor tokens, how
 *             often each dialect was chosen in each dynamic-range bucket and keeping
 *             the most frequent dialect of every bucket.
 *
 * No lookup tables are used anywhere: each rounding searches the 8 magnitudes,
 * each error term is computed from the explicit bin midpoint.
 *
 * Readings taken where the paper is silent (the same list is in the design notes):
 *   - rounding ties (v exactly half-way between two magnitudes) go to the LARGER
 *     magnitude: bins are half-open [k/2,(k+1)/2) and a boundary is the left
 *     edge of its bin (Sec. 3.2: the bin index comes from a shift that drops the low bits);
 *   - dialect ties go to the LOWEST dialect id;
 *   - the exponent is clamped to [exp_min, exp_max]; an all-zero block gets exp_min;
 *   - the sign bit is copied even when the magnitude rounds to 0;
 *   - stage 1: the candidate group is looked up by the bin floor(2*vmax) of the
 *     block maximum (32 entries); by default entry k holds the dialects whose
 *     largest magnitude equals max(8, floor(k/2)); an empty intersection with
 *     the SeDA mask falls back to the SeDA mask alone;
 *   - the residual is the fp32 value of x - xhat (exact for the default exponent
 *     range) and is quantized from that value, never rounded to bf16;
 *   - the scale byte is e + 124, i.e. the E8M0 code of the element scale 2^(e-3);
 *   - sub-formatbook construction: the dynamic-range buckets are the distinct entries
 *     of the stage-1 table; frequency ties (and buckets no anchor block fell into)
 *     go to the lowest dialect id; anchors with an id outside the tensor or a
 *     cluster outside [0, n_clusters) are ignored.
 *
 * Pins (tests/test_oracle_*.py): every representable value of every dialect
 * round-trips; closed form for the uniform dialect; exact-rational brute force
 * on tiny blocks and on all 65536 bf16 patterns; |E_d - exact error| <= G/4;
 * argmin invariant; decomposition never increases any element's error; SeDA
 * choices lie in the mask; per-tile argmax by brute force, the last token of the sequence
 * included; bf16 decode of residual sums against integer round-to-nearest-even (hand-made
 * ties); the residual under a clamped exponent range in exact rationals; sub-formatbooks on
 * hand-counted cases, one dialect per bucket, and a constrained tensor giving
 * back the sub-formatbook it was constrained to; the affine step and the LayerNorm producer in
 * exact rationals (every operation rounded by integer arithmetic, the square root checked by squaring).
 * Parity unpinned: the formatbook VALUES (the paper's table is only in Fig. 2a)
 * and any worked numeric example (the paper prints none).  (The tiled order of the
 * MXFP8 scale bytes is pinned here only by its stated properties; a GPU test hands
 * it to a library block-scaled GEMM.)
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
  int block_size;   /* B: 32 or 16 (any multiple of num_groups up to 64 works here) */
  int num_groups;   /* G: 8, or B */
  int exp_min;      /* clamp of the block exponent e */
  int exp_max;
  int select_mode;  /* 0 = two-stage (Sec. 3.2), 1 = score every allowed dialect */
} fb4o_config;

#define FB4O_MAXB 64

static double bf16_to_double(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  memcpy(&f, &u, 4);
  return (double)f;
}

static int formatbook_ok(const uint8_t *F) {
  for (int d = 0; d < 32; ++d) {
    if (F[d * 8] != 0) return 0;
    for (int j = 1; j < 8; ++j)
      if (F[d * 8 + j] <= F[d * 8 + j - 1] || F[d * 8 + j] > 15) return 0;
  }
  return 1;
}

/* floor(2v) capped at 31: the 0.5-wide bin of a normalised magnitude (Sec. 3.2). */
static int bin_of(double v) {
  double b = floor(2.0 * v);
  return b > 31.0 ? 31 : (int)b;
}

/* index of the magnitude of dialect row Fd nearest to u; ties -> larger magnitude */
static int nearest_index(const uint8_t *Fd, double u) {
  int best = 0;
  double bestd = fabs(u - (double)Fd[0]);
  for (int j = 1; j < 8; ++j) {
    double dj = fabs(u - (double)Fd[j]);
    if (dj <= bestd) { bestd = dj; best = j; }
  }
  return best;
}

/* Default stage-1 table: entry k (bin of the block maximum) -> dialects whose
 * largest magnitude is max(8, k/2)  (Sec. 3.2 two-stage; Sec. 3.4: one bucket per integer block maximum 8..15). */
void fb4o_default_stage1(const uint8_t *F, uint32_t *stage1 /*32*/) {
  for (int k = 0; k < 32; ++k) {
    int bucket = k / 2 < 8 ? 8 : k / 2;
    uint32_t m = 0;
    for (int d = 0; d < 32; ++d)
      if (F[d * 8 + 7] == bucket) m |= 1u << d;
    stage1[k] = m;
  }
}

/* Sec. 3.1: normalised magnitude v = |x| * 2^(3-e), in [0,16) unless the exponent was clamped from above */
static double normalised(double x, int e) { return ldexp(fabs(x), 3 - e); }

/* Sec. 3.1: block exponent e = floor(log2(amax)), clamped; an all-zero block gets exp_min. */
static int block_exponent(double amax, const fb4o_config *cfg) {
  int e;
  if (amax == 0.0) {
    e = cfg->exp_min;
  } else {
    int ex;
    (void)frexp(amax, &ex);          /* amax = m * 2^ex, m in [0.5,1)  =>  floor(log2) = ex-1 */
    e = ex - 1;
    if (e < cfg->exp_min) e = cfg->exp_min;
    if (e > cfg->exp_max) e = cfg->exp_max;
  }
  return e;
}

/*
 * One block.  x[B] are the real input values, sgn[B] their sign bits.
 * allowed = SeDA mask (all ones when unconstrained).
 * Outputs: code[B] (sign<<3 | idx), *did, *e.  If err_q4 != NULL it receives,
 * for every dialect, the approximate error in quarter units (-1 for dialects
 * that were not candidates).
 */
static void quantize_block(const double *x, const uint8_t *sgn, const fb4o_config *cfg,
                           const uint8_t *F, const uint32_t *stage1, uint32_t allowed,
                           uint8_t *code, int *did, int *e_out, int32_t *err_q4) {
  const int B = cfg->block_size, G = cfg->num_groups, gs = B / G;
  /* Sec. 3.1: shared power-of-two scale from floor(log2(max magnitude)) */
  double amax = 0.0;
  for (int i = 0; i < B; ++i) if (fabs(x[i]) > amax) amax = fabs(x[i]);
  const int e = block_exponent(amax, cfg);
  /* normalise: v = |x| * 2^(3-e), in [0,16) unless the exponent was clamped from above */
  double v[FB4O_MAXB];
  for (int i = 0; i < B; ++i) v[i] = normalised(x[i], e);
  /* Sec. 3.2: group-wise maxima */
  double gmax[FB4O_MAXB];
  double vmax = 0.0;
  for (int g = 0; g < G; ++g) {
    double m = 0.0;
    for (int i = 0; i < gs; ++i) if (v[g * gs + i] > m) m = v[g * gs + i];
    gmax[g] = m;
    if (m > vmax) vmax = m;
  }
  /* stage 1: sub-formatbook by the block maximum, intersected with the SeDA set */
  uint32_t cand = allowed;
  if (cfg->select_mode == 0) {
    cand = stage1[bin_of(vmax)] & allowed;
    if (cand == 0) cand = allowed;
  }
  /* stage 2: approximate error = sum over group maxima of |bin midpoint - nearest value| */
  int best = -1;
  double best_err = 0.0;
  for (int d = 0; d < 32; ++d) {
    if (err_q4) err_q4[d] = -1;
    if (!((cand >> d) & 1u)) continue;
    double err = 0.0;
    for (int g = 0; g < G; ++g) {
      double mid = 0.5 * (double)bin_of(gmax[g]) + 0.25;
      err += fabs(mid - (double)F[d * 8 + nearest_index(F + d * 8, mid)]);
    }
    if (err_q4) err_q4[d] = (int32_t)(4.0 * err);
    if (best < 0 || err < best_err) { best = d; best_err = err; }   /* ties keep the lowest id */
  }
  /* quantize every element to the nearest magnitude of the chosen dialect */
  for (int i = 0; i < B; ++i)
    code[i] = (uint8_t)((sgn[i] << 3) | nearest_index(F + best * 8, v[i]));
  *did = best;
  *e_out = e;
}

static double dequant_value(const uint8_t *F, int did, int e, uint8_t code) {
  double mag = ldexp((double)F[did * 8 + (code & 7)], e - 3);
  return (code & 8) ? -mag : mag;
}

static void store_block(const uint8_t *code, int B, int did, int e, uint8_t *codes_row, uint16_t *meta_row,
                        int64_t blk) {
  for (int i = 0; i < B; i += 2)
    codes_row[(blk * B + i) / 2] = (uint8_t)(code[i] | (code[i + 1] << 4));
  meta_row[blk] = (uint16_t)((e + 124) | (did << 8));
}

static int config_ok(const fb4o_config *cfg, int64_t C) {
  if (cfg->block_size <= 0 || cfg->block_size > FB4O_MAXB || (cfg->block_size & 1)) return 0;
  if (cfg->num_groups <= 0 || cfg->block_size % cfg->num_groups) return 0;
  if (cfg->exp_min < -124 || cfg->exp_max > 127 || cfg->exp_min > cfg->exp_max) return 0;
  if (C <= 0 || C % cfg->block_size) return 0;
  return 1;
}

static uint32_t row_mask(const int32_t *cluster_id, const uint32_t *cluster_mask, int32_t n_clusters, int64_t t) {
  if (!cluster_id || cluster_id[t] < 0) return 0xffffffffu;
  if (cluster_id[t] >= n_clusters) return 0;   /* caller error; reported by the entry points */
  return cluster_mask[cluster_id[t]];
}

/* Salient-token set, Sec. 3.3: the highest-scoring token of every tile of `tile`
 * consecutive tokens (ties -> lowest index); ascending list; returns its length. */
int64_t fb4o_select_salient(const float *score, int64_t T, int32_t tile, int32_t *salient_idx) {
  if (tile <= 0 || T < 0) return -1;
  int64_t n = 0;
  for (int64_t t0 = 0; t0 < T; t0 += tile) {
    int64_t t1 = t0 + tile < T ? t0 + tile : T, arg = t0;
    for (int64_t t = t0 + 1; t < t1; ++t) if (score[t] > score[arg]) arg = t;
    salient_idx[n++] = (int32_t)arg;
  }
  return n;
}

/* The other reading of "salient tokens = the top 5 % by score": the k highest-scoring tokens of the
 * whole sequence (ties -> lowest index), listed in ascending token order.  Plain selection sort of
 * the candidates, k rounds. */
int64_t fb4o_select_salient_topk(const float *score, int64_t T, int64_t k, int32_t *salient_idx) {
  if (T < 0 || k < 0 || k > T) return -1;
  uint8_t *taken = (uint8_t *)calloc((size_t)(T > 0 ? T : 1), 1);
  if (!taken) return -1;
  for (int64_t r = 0; r < k; ++r) {
    int64_t arg = -1;
    for (int64_t t = 0; t < T; ++t)
      if (!taken[t] && (arg < 0 || score[t] > score[arg])) arg = t;   /* first maximum = lowest index */
    if (arg < 0) break;   /* cannot happen (k <= T): keeps the compiler's bounds analysis quiet */
    taken[arg] = 1;
  }
  int64_t n = 0;
  for (int64_t t = 0; t < T; ++t) if (taken[t]) salient_idx[n++] = (int32_t)t;
  free(taken);
  return n;
}

/*
 * Quantize a T x C bf16 tensor (bit patterns, `ld` elements between rows).
 * Optional SeDA tables (cluster_id NULL => unconstrained).  Optional residual
 * pass for the rows listed (ascending) in salient_idx: residual codes/meta are
 * written compactly, row s of res_* belonging to token salient_idx[s].
 * err_q4 (optional, T*C/B*32 int32) receives the per-dialect approximate errors
 * of the main pass.
 * Returns 0, or a negative code for invalid arguments.
 */
int fb4o_quantize(const uint16_t *x, int64_t T, int64_t C, int64_t ld,
                  const fb4o_config *cfg, const uint8_t *F, const uint32_t *stage1_in,
                  const int32_t *cluster_id, const uint32_t *cluster_mask, int32_t n_clusters,
                  const int32_t *salient_idx, int64_t n_salient,
                  uint8_t *codes, uint16_t *meta, uint8_t *res_codes, uint16_t *res_meta,
                  int32_t *err_q4) {
  if (!config_ok(cfg, C) || T < 0 || ld < C) return -1;
  if (!formatbook_ok(F)) return -2;
  uint32_t stage1[32];
  if (stage1_in) memcpy(stage1, stage1_in, sizeof stage1); else fb4o_default_stage1(F, stage1);
  const int B = cfg->block_size;
  const int64_t nblk = C / B;
  int bad = 0;
  if (cluster_id)
    for (int64_t t = 0; t < T; ++t)
      if (cluster_id[t] >= n_clusters || (cluster_id[t] >= 0 && cluster_mask[cluster_id[t]] == 0)) bad = 1;
  for (int64_t s = 0; s < n_salient; ++s) {
    if (salient_idx[s] < 0 || salient_idx[s] >= T) bad = 1;
    if (s > 0 && salient_idx[s] <= salient_idx[s - 1]) bad = 1;
  }
  if (bad) return -3;

#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < T; ++t) {
    const uint32_t allowed = row_mask(cluster_id, cluster_mask, n_clusters, t);
    /* is this row salient?  (ascending list => binary search) */
    int64_t srow = -1;
    {
      int64_t lo = 0, hi = n_salient - 1;
      while (lo <= hi) {
        int64_t mid = (lo + hi) / 2;
        if (salient_idx[mid] == t) { srow = mid; break; }
        if (salient_idx[mid] < t) lo = mid + 1; else hi = mid - 1;
      }
    }
    for (int64_t blk = 0; blk < nblk; ++blk) {
      double xv[FB4O_MAXB];
      uint8_t sg[FB4O_MAXB], code[FB4O_MAXB];
      for (int i = 0; i < B; ++i) {
        uint16_t b = x[t * ld + blk * B + i];
        xv[i] = bf16_to_double(b);
        sg[i] = (uint8_t)(b >> 15);
      }
      int did, e;
      quantize_block(xv, sg, cfg, F, stage1, allowed, code, &did, &e,
                     err_q4 ? err_q4 + (t * nblk + blk) * 32 : NULL);
      store_block(code, B, did, e, codes + t * (C / 2), meta + t * nblk, blk);
      if (srow >= 0) {
        /* Sec. 3.3: Act = Q(Act) + Delta; quantize Delta again with the same candidate set */
        double dv[FB4O_MAXB];
        uint8_t dsg[FB4O_MAXB], dcode[FB4O_MAXB];
        for (int i = 0; i < B; ++i) {
          float df = (float)(xv[i] - dequant_value(F, did, e, code[i]));
          dv[i] = (double)df;
          dsg[i] = (uint8_t)(signbit(df) ? 1 : 0);
        }
        int rdid, re;
        quantize_block(dv, dsg, cfg, F, stage1, allowed, dcode, &rdid, &re, NULL);
        store_block(dcode, B, rdid, re, res_codes + srow * (C / 2), res_meta + srow * nblk, blk);
      }
    }
  }
  return 0;
}

/*
 * The same quantization for float32 input (a producer handing over its fp32 result, App. D.2
 * fusion with the preceding operation): every value is taken as it is, nothing is rounded to
 * bf16 first.  Optional SeDA tables as in fb4o_quantize (Sec. 3.4); no residual pass.
 */
int fb4o_quantize_f32(const float *x, int64_t T, int64_t C, int64_t ld, const fb4o_config *cfg,
                      const uint8_t *F, const uint32_t *stage1_in,
                      const int32_t *cluster_id, const uint32_t *cluster_mask, int32_t n_clusters,
                      uint8_t *codes, uint16_t *meta) {
  if (!config_ok(cfg, C) || T < 0 || ld < C) return -1;
  if (!formatbook_ok(F)) return -2;
  uint32_t stage1[32];
  if (stage1_in) memcpy(stage1, stage1_in, sizeof stage1); else fb4o_default_stage1(F, stage1);
  const int B = cfg->block_size;
  const int64_t nblk = C / B;
  if (cluster_id)
    for (int64_t t = 0; t < T; ++t)
      if (cluster_id[t] >= n_clusters || (cluster_id[t] >= 0 && cluster_mask[cluster_id[t]] == 0)) return -3;
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < T; ++t) {
    /* Sec. 3.4: the token's sub-formatbook restricts the candidates, whatever the input type */
    const uint32_t allowed = row_mask(cluster_id, cluster_mask, n_clusters, t);
    for (int64_t blk = 0; blk < nblk; ++blk) {
      double xv[FB4O_MAXB];
      uint8_t sg[FB4O_MAXB], code[FB4O_MAXB];
      for (int i = 0; i < B; ++i) {
        float f = x[t * ld + blk * B + i];
        xv[i] = (double)f;
        sg[i] = (uint8_t)(signbit(f) ? 1 : 0);
      }
      int did, e;
      quantize_block(xv, sg, cfg, F, stage1, allowed, code, &did, &e, NULL);
      store_block(code, B, did, e, codes + t * (C / 2), meta + t * nblk, blk);
    }
  }
  return 0;
}

/*
 * Per-channel affine producer in front of the quantizer (App. D.2: quantization is fused with the
 * preceding operation, e.g. LayerNorm; the elementwise tail of a LayerNorm is y = x * gamma_c +
 * beta_c, and the modulation of Open-Sora 2.0's blocks, Sec. 3.3, is y = x * (1 + scale_c) +
 * shift_c):  y[t][c] = x[t][c] * g_c + bias_c  with  g_c = gain_c  or  1 + gain_c (plus_one),
 * x, gain and bias given as bf16.  The arithmetic is float32 as in the fused kernel, stated
 * exactly: g_c is the float32 nearest to 1 + gain_c, and y is the float32 nearest to the exact
 * value of x * g_c + bias_c (one rounding: fmaf).  The result feeds fb4o_quantize_f32.
 */
int fb4o_affine_f32(const uint16_t *x, int64_t T, int64_t C, int64_t ld, const uint16_t *gain,
                    const uint16_t *bias, int plus_one, float *y) {
  if (T < 0 || C <= 0 || ld < C) return -1;
  for (int64_t t = 0; t < T; ++t) {
    for (int64_t c = 0; c < C; ++c) {
      const float xf = (float)bf16_to_double(x[t * ld + c]);
      float g = (float)bf16_to_double(gain[c]);
      const float b = (float)bf16_to_double(bias[c]);
      if (plus_one) g = 1.0f + g;
      y[t * C + c] = fmaf(xf, g, b);
    }
  }
  return 0;
}

/*
 * LayerNorm with per-channel modulation in front of the quantizer (App. D.2 names LayerNorm as an operation
 * the quantizer is fused behind; in the adaLN blocks the normalised activation is modulated as
 * y = n * (1 + scale_c) + shift_c before the linear layer).  Per token, in float32, with every operation
 * rounded once (IEEE binary32, round to nearest even) and the order of the additions stated:
 *   block sums    s_b = (((x_0 + x_1) + x_2) + ...) over the 32 consecutive channels of block b;
 *   segment sums  the block sums of 32 consecutive blocks (1024 channels; a short last segment is filled
 *                 up with +0) are added as a butterfly: for off = 16, 8, 4, 2, 1, all at once,
 *                 v_i <- v_i + v_(i xor off); the segment sum is v_0;
 *   row total     the segment sums added to +0 in order, (((0 + S_0) + S_1) + S_2) + ...;
 *   mean = total / C;  d_i = x_i - mean;
 *   the sum of squares by the same three steps with q_b = fma(d, d, q) over the block's channels in order
 *   (q = 0 at the start);  var = total of squares / C;  rstd = 1 / sqrt(var + eps);
 *   y_i = fma(d_i * rstd, g_c, bias_c),  g_c = gain_c or 1 + gain_c (float32 sum).
 * x, gain, bias are bf16 bit patterns; y feeds fb4o_quantize_f32.  C must be a multiple of 32.
 */
static float ln_segment_butterfly(const float *blocksum, int n) {
  float v[32], u[32];
  for (int i = 0; i < 32; ++i) v[i] = i < n ? blocksum[i] : 0.0f;
  for (int off = 16; off >= 1; off >>= 1) {
    for (int i = 0; i < 32; ++i) u[i] = v[i] + v[i ^ off];
    memcpy(v, u, sizeof v);
  }
  return v[0];
}

static float ln_row_total(const float *blocksum, int64_t nblk) {
  float total = 0.0f;
  for (int64_t b0 = 0; b0 < nblk; b0 += 32) {
    int n = nblk - b0 < 32 ? (int)(nblk - b0) : 32;
    total = total + ln_segment_butterfly(blocksum + b0, n);
  }
  return total;
}

int fb4o_layernorm_f32(const uint16_t *x, int64_t T, int64_t C, int64_t ld, const uint16_t *gain,
                       const uint16_t *bias, int plus_one, float eps, float *y, float *stats /* optional [T][2]: mean, var */) {
  if (T < 0 || C <= 0 || C % 32 || ld < C) return -1;
  const int64_t nblk = C / 32;
  float *bs = (float *)malloc((size_t)nblk * sizeof(float));
  float *d = (float *)malloc((size_t)C * sizeof(float));
  if (!bs || !d) { free(bs); free(d); return -1; }
  for (int64_t t = 0; t < T; ++t) {
    for (int64_t b = 0; b < nblk; ++b) {
      float s = (float)bf16_to_double(x[t * ld + b * 32]);
      for (int i = 1; i < 32; ++i) s = s + (float)bf16_to_double(x[t * ld + b * 32 + i]);
      bs[b] = s;
    }
    const float mean = ln_row_total(bs, nblk) / (float)C;
    for (int64_t b = 0; b < nblk; ++b) {
      float q = 0.0f;
      for (int i = 0; i < 32; ++i) {
        float di = (float)bf16_to_double(x[t * ld + b * 32 + i]) - mean;
        d[b * 32 + i] = di;
        q = fmaf(di, di, q);
      }
      bs[b] = q;
    }
    const float var = ln_row_total(bs, nblk) / (float)C;
    const float rstd = 1.0f / sqrtf(var + eps);
    if (stats) { stats[2 * t] = mean; stats[2 * t + 1] = var; }
    for (int64_t c = 0; c < C; ++c) {
      float g = (float)bf16_to_double(gain[c]);
      const float bc = (float)bf16_to_double(bias[c]);
      if (plus_one) g = 1.0f + g;
      y[t * C + c] = fmaf(d[c] * rstd, g, bc);
    }
  }
  free(bs);
  free(d);
  return 0;
}

static uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  return (uint16_t)(u >> 16);
}

/*
 * Decode: xhat = (-1)^s * F[did][idx] * 2^(e-3); salient rows add the decoded
 * residual, the sum being rounded once to fp32.  out_dtype 0: float32 out,
 * 1: bf16 bit patterns (round-to-nearest-even of the fp32 result),
 * 2: IEEE half bit patterns (the compiler's float -> _Float16 conversion: round to
 *    nearest even, overflow to infinity), the type the paper's H100 pipeline decodes to (App. D.2).
 */
int fb4o_dequantize(const uint8_t *codes, const uint16_t *meta, int64_t T, int64_t C, int block_size,
                    const uint8_t *F, const int32_t *salient_idx, int64_t n_salient,
                    const uint8_t *res_codes, const uint16_t *res_meta, void *out, int out_dtype) {
  if (block_size <= 0 || C % block_size || !formatbook_ok(F)) return -1;
  const int B = block_size;
  const int64_t nblk = C / B;
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < T; ++t) {
    int64_t srow = -1;
    for (int64_t s = 0; s < n_salient; ++s) if (salient_idx[s] == t) { srow = s; break; }
    for (int64_t c = 0; c < C; ++c) {
      int64_t blk = c / B;
      uint16_t m = meta[t * nblk + blk];
      uint8_t byte = codes[t * (C / 2) + c / 2];
      uint8_t code = (c & 1) ? (byte >> 4) : (byte & 15);
      float val = (float)dequant_value(F, m >> 8, (int)(m & 0xff) - 124, code);
      if (srow >= 0) {
        uint16_t rm = res_meta[srow * nblk + blk];
        uint8_t rb = res_codes[srow * (C / 2) + c / 2];
        uint8_t rc = (c & 1) ? (rb >> 4) : (rb & 15);
        double r = dequant_value(F, rm >> 8, (int)(rm & 0xff) - 124, rc);
        val = (float)((double)val + r);
      }
      if (out_dtype == 0) {
        ((float *)out)[t * C + c] = val;
      } else if (out_dtype == 1) {
        ((uint16_t *)out)[t * C + c] = f32_to_bf16_rne(val);
      } else {
        _Float16 h = (_Float16)val;
        memcpy((uint16_t *)out + t * C + c, &h, 2);
      }
    }
  }
  return 0;
}

/* mean squared error between the bf16 input and a reconstruction, accumulated in fp64 */
double fb4o_mse(const uint16_t *x, int64_t ld, const float *recon, int64_t T, int64_t C) {
  double acc = 0.0;
  for (int64_t t = 0; t < T; ++t) {
    double row = 0.0;
    for (int64_t c = 0; c < C; ++c) {
      double d = bf16_to_double(x[t * ld + c]) - (double)recon[t * C + c];
      row += d * d;
    }
    acc += row;
  }
  return T * C ? acc / ((double)T * (double)C) : 0.0;
}

/*
 * One block given as doubles (for pins and brute-force comparisons on values
 * that are not bf16, e.g. residuals).  code[B], err_q4[32] may be inspected.
 */
int fb4o_quantize_block_f64(const double *x, const fb4o_config *cfg, const uint8_t *F,
                            const uint32_t *stage1_in, uint32_t allowed,
                            uint8_t *code, int32_t *did, int32_t *e, int32_t *err_q4) {
  if (!config_ok(cfg, cfg->block_size) || !formatbook_ok(F) || allowed == 0) return -1;
  uint32_t stage1[32];
  if (stage1_in) memcpy(stage1, stage1_in, sizeof stage1); else fb4o_default_stage1(F, stage1);
  uint8_t sg[FB4O_MAXB];
  for (int i = 0; i < cfg->block_size; ++i) sg[i] = (uint8_t)(signbit(x[i]) ? 1 : 0);
  int d_, e_;
  quantize_block(x, sg, cfg, F, stage1, allowed, code, &d_, &e_, err_q4);
  *did = d_;
  *e = e_;
  return 0;
}

/*
 * Sub-formatbook construction, Sec. 3.4 (a histogram of the dialects chosen on a cluster's anchor
 * tokens; every dynamic-range bucket keeps its most frequent member).
 * meta [T][nblk] holds the dialect chosen for every block (bits 8-12).  Anchor a is
 * token anchor_token[a] and belongs to cluster anchor_cluster[a].  For every cluster:
 * count how often each dialect occurs in the blocks of its anchor tokens; then, for
 * every dynamic-range bucket (a distinct entry of the stage-1 table), keep the most
 * frequent dialect among the bucket's members.  cluster_mask[c] = the kept dialects.
 */
int fb4o_build_subformatbook(const uint16_t *meta, int64_t T, int64_t nblk,
                             const int32_t *anchor_token, const int32_t *anchor_cluster, int64_t n_anchor,
                             int32_t n_clusters, const uint8_t *F, const uint32_t *stage1_in,
                             uint32_t *cluster_mask) {
  if (T < 0 || nblk <= 0 || n_anchor < 0 || n_clusters < 0 || !formatbook_ok(F)) return -1;
  uint32_t stage1[32];
  if (stage1_in) memcpy(stage1, stage1_in, sizeof stage1); else fb4o_default_stage1(F, stage1);
  for (int32_t c = 0; c < n_clusters; ++c) {
    int64_t count[32];
    for (int d = 0; d < 32; ++d) count[d] = 0;
    for (int64_t a = 0; a < n_anchor; ++a) {
      if (anchor_cluster[a] != c) continue;
      int64_t t = anchor_token[a];
      if (t < 0 || t >= T) continue;
      for (int64_t b = 0; b < nblk; ++b) count[(meta[t * nblk + b] >> 8) & 31] += 1;
    }
    uint32_t mask = 0;
    for (int k = 0; k < 32; ++k) {            /* every bucket; repeated entries pick the same dialect again */
      int best = -1;
      for (int d = 0; d < 32; ++d) {
        if (!((stage1[k] >> d) & 1u)) continue;
        if (best < 0 || count[d] > count[best]) best = d;   /* ties keep the lowest id */
      }
      if (best >= 0) mask |= 1u << best;
    }
    cluster_mask[c] = mask;
  }
  return 0;
}

/*
 * MXFP8 view of a quantized tensor (App. D.2: the integer magnitudes 0..15 are all e4m3 numbers
 * and the block scale is a power of two, which makes an FB4 tensor an MXFP8 operand without any
 * rounding).  Every element becomes the e4m3 byte of its signed integer magnitude
 * (sign, 4-bit exponent with bias 7, 3-bit mantissa), every 32-element block gets the E8M0 byte
 * of its element scale 2^(e-3), which is the block's scale byte itself (E8M0 of 2^k is k+127).
 *
 * Scale layouts: 0 = row-major [T][C/32].  1 = tiles of 128 rows x 4 scale columns, 512 bytes
 * each, the tiles of a row band stored one after the other (column tiles contiguous); inside a
 * tile the scale of (row r, column c) sits at (r mod 32)*16 + (r div 32)*4 + c.  This is the
 * arrangement block-scaled tensor-core GEMMs on Blackwell read their scale factors in; rows are
 * padded to a multiple of 128 and scale columns to a multiple of 4, padding entries hold 0x7f
 * (scale 1).
 */
int64_t fb4o_mxfp8_scale_offset(int64_t row, int64_t col, int64_t n_col, int layout) {
  if (layout == 0) return row * n_col + col;
  int64_t col_tiles = (n_col + 3) / 4;
  int64_t tile = (row / 128) * col_tiles + col / 4;
  int64_t r = row % 128;
  return tile * 512 + (r % 32) * 16 + (r / 32) * 4 + col % 4;
}

int64_t fb4o_mxfp8_scale_bytes(int64_t T, int64_t C, int layout) {
  int64_t n_col = C / 32;
  if (layout == 0) return T * n_col;
  return ((T + 127) / 128) * ((n_col + 3) / 4) * 512;
}

static uint8_t e4m3_of_small_int(int m) {   /* m in 0..15, exact */
  if (m == 0) return 0;
  int ex = 0;
  while ((m >> (ex + 1)) != 0) ++ex;               /* floor(log2 m) */
  int frac = m - (1 << ex);                          /* m = 2^ex * (1 + frac / 2^ex) */
  int mant = ex <= 3 ? frac << (3 - ex) : frac >> (ex - 3);
  return (uint8_t)(((ex + 7) << 3) | mant);
}

int fb4o_to_mxfp8(const uint8_t *codes, const uint16_t *meta, int64_t T, int64_t C, const uint8_t *F,
                  uint8_t *e4m3, uint8_t *scales, int layout) {
  if (C <= 0 || C % 32 || T < 0 || !formatbook_ok(F) || (layout != 0 && layout != 1)) return -1;
  const int64_t nblk = C / 32;
  memset(scales, 0x7f, (size_t)fb4o_mxfp8_scale_bytes(T, C, layout));
  for (int64_t t = 0; t < T; ++t) {
    for (int64_t c = 0; c < C; ++c) {
      uint16_t m = meta[t * nblk + c / 32];
      uint8_t byte = codes[t * (C / 2) + c / 2];
      uint8_t code = (c & 1) ? (byte >> 4) : (byte & 15);
      e4m3[t * C + c] = (uint8_t)(e4m3_of_small_int(F[(m >> 8) * 8 + (code & 7)]) | ((code & 8) << 4));
    }
    for (int64_t b = 0; b < nblk; ++b)
      scales[fb4o_mxfp8_scale_offset(t, b, nblk, layout)] = (uint8_t)(meta[t * nblk + b] & 0xff);
  }
  return 0;
}

/*
 * Offline weight quantization (Sec. 3.3: weights are available before inference, so every dialect
 * can be tried on every element; App. C: the squared error decides).  Per block: the same power-of-two scale as for
 * activations; then for EVERY dialect the squared error of rounding every element to its nearest
 * magnitude, summed over the block's elements in index order in double precision (each term
 * (v - m)^2 is exact in double; only the running sum rounds); the dialect with the smallest sum
 * wins, ties to the lowest id; the elements are rounded with it.  No groups, no stage 1, no tables.
 * sse (optional, [N*K/B][32]) receives the sums.
 */
int fb4o_quantize_weights(const uint16_t *w, int64_t N, int64_t K, int64_t ld, const fb4o_config *cfg,
                          const uint8_t *F, uint8_t *codes, uint16_t *meta, double *sse) {
  if (!config_ok(cfg, K) || N < 0 || ld < K) return -1;
  if (!formatbook_ok(F)) return -2;
  const int B = cfg->block_size;
  const int64_t nblk = K / B;
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < N; ++n) {
    for (int64_t blk = 0; blk < nblk; ++blk) {
      double x[FB4O_MAXB], v[FB4O_MAXB];
      uint8_t sg[FB4O_MAXB], code[FB4O_MAXB];
      double amax = 0.0;
      for (int i = 0; i < B; ++i) {
        uint16_t b = w[n * ld + blk * B + i];
        x[i] = bf16_to_double(b);
        sg[i] = (uint8_t)(b >> 15);
        if (fabs(x[i]) > amax) amax = fabs(x[i]);
      }
      const int e = block_exponent(amax, cfg);
      for (int i = 0; i < B; ++i) v[i] = normalised(x[i], e);
      int best = 0;
      double best_err = 0.0;
      for (int d = 0; d < 32; ++d) {
        double err = 0.0;
        for (int i = 0; i < B; ++i) {
          double diff = v[i] - (double)F[d * 8 + nearest_index(F + d * 8, v[i])];
          err += diff * diff;
        }
        if (sse) sse[(n * nblk + blk) * 32 + d] = err;
        if (d == 0 || err < best_err) { best = d; best_err = err; }
      }
      for (int i = 0; i < B; ++i)
        code[i] = (uint8_t)((sg[i] << 3) | nearest_index(F + best * 8, v[i]));
      store_block(code, B, best, e, codes + n * (K / 2), meta + n * nblk, blk);
    }
  }
  return 0;
}
