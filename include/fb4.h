/*
 * fb4.h -- C ABI of the B200 (sm_100a) FB4 online activation quantizer.
 *
 * FB4 is the 4-bit block format of SemanticDialect: every block of B contiguous
 * channels of a token shares a power-of-two scale and one of 32 "dialects"
 * (8 integer magnitudes out of 0..15); an element is a sign bit plus a 3-bit
 * index into the block's dialect (Sec. 3.1).  The dialect is chosen online, per
 * block, by summing a lookup-table estimate of the quantization error over the
 * block's group-wise maxima and taking the minimum inside the sub-formatbook
 * that matches the block's dynamic range (Sec. 3.2).
 *
 * Conventions for every call
 *   - Return value: FB4_OK (0) or a negative FB4_ERR_* code.  Nothing is printed,
 *     nothing aborts.  fb4_strerror() names a code.
 *   - Unless a parameter says "host", data pointers are DEVICE pointers owned by
 *     the caller; the library never frees or retains them.  The library owns only
 *     the opaque context (a few KB of lookup tables on the device).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls enqueue work on it and return without synchronising; launch errors
 *     that CUDA reports synchronously come back as FB4_ERR_CUDA.
 *   - Tensors are row-major [T tokens][C channels]; blocks run along the
 *     contiguous channel axis.  C must be a multiple of the block size.
 *     `ld_elems` is the distance between rows of x in elements (>= C).
 *   - x is bfloat16.  Inputs must be finite (NaN/Inf are not checked and give
 *     meaningless, but in-bounds, output).
 *   - Alignment: x and every output pointer must be 16-byte aligned and
 *     ld_elems a multiple of 8; otherwise FB4_ERR_ALIGN.
 *   - The device of the context must be the current device of the calling thread.
 *   - Host threads: a context is not internally locked.  Calls on ONE context must be serialised by
 *     the caller (the context keeps a launch counter, the name of the last kernel variant, the
 *     staging streams of fb4_quantize_host and scratch of the global top-k selection, all unguarded).
 *     Different contexts, also on the same device, may be used from different threads at the
 *     same time; one-time library set-up (driver entry points, the address of the built-in
 *     scratch of the *_static call) is guarded inside the library.  fb4_init / fb4_destroy of
 *     different contexts may run concurrently.
 *   - Device code has no unbounded wait loops: the only waits (for asynchronous loads into
 *     shared memory) give up after a fixed number of tries and raise a status bit
 *     (fb4_device_status); a call cannot hang.
 *
 * Output layout
 *   codes : uint8 [T][C/2].  Byte j of a row holds element 2j in its low nibble
 *           and element 2j+1 in its high nibble; nibble = sign<<3 | index.
 *   meta  : uint16 [T][C/B].  bits 0-7 = scale byte = e + 124 where e is the
 *           block exponent floor(log2(amax)) (clamped); this is the E8M0 code of
 *           the element scale 2^(e-3).  bits 8-12 = dialect id.  bits 13-15 = 0.
 *   value : (-1)^sign * formatbook[dialect][index] * 2^(e-3).
 */
#ifndef FB4_H_
#define FB4_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FB4_OK 0
#define FB4_ERR_INVALID_ARG (-1) /* null pointer, bad enum, negative count, empty dialect mask */
#define FB4_ERR_SHAPE (-2)       /* C not a multiple of the block size, ld_elems < C, T < 0 */
#define FB4_ERR_ALIGN (-3)       /* pointer not 16-byte aligned or ld_elems not a multiple of 8 */
#define FB4_ERR_FORMATBOOK (-4)  /* dialect not strictly ascending from 0 within 0..15 */
#define FB4_ERR_CUDA (-5)        /* a CUDA runtime call failed; fb4_last_cuda_error() has the code */
#define FB4_ERR_NO_DEVICE (-6)   /* no usable CUDA device / wrong architecture (needs sm_100) */
#define FB4_ERR_STATIC_LIMIT (-7) /* more clusters than the built-in scratch of a *_static call holds */

typedef struct fb4_ctx fb4_ctx;

/* Quantizer parameters (Sec. 4.1: block sizes 16 and 32, num_groups = 8 by default;
 * Table 2 also evaluates num_groups = block size). */
typedef struct {
  uint32_t block_size;  /* 32 (default) or 16 */
  uint32_t num_groups;  /* 8 (default) or block_size; contiguous groups of block_size/num_groups */
  int32_t exp_min;      /* clamp of the block exponent e; default -124 (>= -124) */
  int32_t exp_max;      /* default 127 (<= 127); the paper's 5-bit exponent is e.g. [-15,16] */
  uint32_t select_mode; /* 0 = two-stage selection (Sec. 3.2); 1 = score every allowed dialect */
} fb4_config;

/* Defaults: {32, 8, -124, 127, 0}. */
void fb4_default_config(fb4_config* cfg);

/*
 * Build a context on CUDA device `device`: validates the formatbook, builds the
 * Qvalue / Qerror lookup tables (Sec. 3.2: 0.5-wide bins; Qvalue = exact index of
 * the nearest magnitude, Qerror = absolute error at the bin midpoint) and the
 * stage-1 table, and uploads them.  Synchronous; may allocate device memory.
 *   formatbook  : host, 32*8 bytes, dialect-major; NULL = the built-in stand-in
 *                 table (the paper gives its table only as Fig. 2a).
 *   stage1_mask : host, 32 words; entry k = bit mask of the dialects compared when
 *                 the block maximum falls in bin k = floor(2*vmax) (Sec. 3.2:
 *                 stage 1 of the two-stage selection).  NULL = dialects
 *                 whose largest magnitude equals max(8, k/2).
 *   cfg         : NULL = defaults.
 * On success *out owns device memory until fb4_destroy().
 */
int fb4_init(fb4_ctx** out, int device, const uint8_t* formatbook, const uint32_t* stage1_mask,
             const fb4_config* cfg);
int fb4_destroy(fb4_ctx* ctx);

/* Host copies of the tables a context was built with (any pointer may be NULL):
 * formatbook[32*8], stage1_mask[32], qvalue[32 dialects][32 bins] (index 0..7),
 * qerror_q4[32][32] (error in quarter units).  For tests and diagnostics. */
int fb4_get_tables(const fb4_ctx* ctx, uint8_t* formatbook, uint32_t* stage1_mask, uint8_t* qvalue,
                   uint8_t* qerror_q4);

/*
 * The table image that the device code of include/fb4_block.cuh reads (App. D.2: the quantizer as the
 * tail of a producer kernel; that header holds the per-block routine the library's own kernels use).
 * *device_image receives a DEVICE pointer owned by the context (valid until fb4_destroy), *bytes its
 * size (= sizeof(fb4blk::Tables)).  FB4_ERR_INVALID_ARG if the context's configuration is not the one
 * the header implements (block 32, 8 groups, two-stage selection, full exponent range) or its
 * formatbook / stage-1 table does not fit the packed layout.
 */
int fb4_block_tables(const fb4_ctx* ctx, const void** device_image, uint64_t* bytes);

/*
 * Plain FB4 quantization of x[T][C] (Sec. 3.1-3.2): per block, scale -> group
 * maxima -> LUT error sums over the stage-1 candidates -> argmin (ties: lowest
 * dialect id) -> LUT quantization.  Writes codes[T][C/2] and meta[T][C/B].
 * T == 0 is a no-op.
 */
int fb4_quantize(fb4_ctx* ctx, const void* x_bf16, int64_t T, int64_t C, int64_t ld_elems, uint8_t* codes,
                 uint16_t* meta, void* stream);

/*
 * fb4_quantize for float32 input (App. D.2 runs the quantizer as the tail of the operation in
 * front of it, an activation function or a normalisation: a producer that still holds its result
 * in fp32 hands it over without rounding it to bf16 first).  The values are quantized as they are: the block
 * exponent is the fp32 exponent of the largest magnitude, bins come from the full fp32 mantissa.
 *   x : device float32 [T][ld_elems], finite; 16-byte aligned, ld_elems a multiple of 4
 */
int fb4_quantize_f32(fb4_ctx* ctx, const float* x, int64_t T, int64_t C, int64_t ld_elems, uint8_t* codes,
                     uint16_t* meta, void* stream);

/*
 * A per-channel affine producer fused in front of the quantizer (App. D.2: quantization is fused
 * with the preceding operation such as LayerNorm; the elementwise tail of a LayerNorm is
 * y = x * gamma_c + beta_c, the modulation in front of the linear layers of an adaLN block is
 * y = x * (1 + scale_c) + shift_c):
 *     y[t][c] = x[t][c] * g_c + bias_c,   g_c = gain_c (gain_plus_one 0) or 1 + gain_c (1),
 * evaluated in float32 exactly as stated - g_c is the float32 nearest to 1 + gain_c, y the float32
 * nearest to the exact x * g_c + bias_c (one fused multiply-add) - and quantized from registers as
 * fb4_quantize_f32 quantizes a float32 tensor; y is never rounded to bfloat16 and never stored.
 * Optional SeDA restriction as in fb4_quantize_seda (Sec. 3.4; the layers the paper applies SeDA to sit
 * behind such a producer); no residual pass.  The default configuration with C a multiple of 64
 * runs in one TMA-staged pass at 2.56 bytes per element; any other configuration runs in the
 * generic kernel with the same result.
 *   x    : device bfloat16 [T][ld_elems]
 *   gain : device bfloat16 [C];  bias : device bfloat16 [C]   (per channel, shared by all tokens)
 *   cluster_id : NULL = unconstrained (then cluster_mask is ignored); else as in fb4_quantize_seda
 */
int fb4_quantize_affine(fb4_ctx* ctx, const void* x_bf16, int64_t T, int64_t C, int64_t ld_elems,
                        const void* gain_bf16, const void* bias_bf16, int gain_plus_one,
                        const int32_t* cluster_id, const uint32_t* cluster_mask, int32_t n_clusters,
                        uint8_t* codes, uint16_t* meta, void* stream);

/*
 * fb4_quantize_affine with the result written as an MXFP8 operand (App. D.2): producer, quantizer
 * and MXFP8 view in one pass - bf16 in, e4m3 bytes + E8M0 scales out, 3.03 bytes per element, and
 * neither y nor the 4-bit codes reach memory.  The output equals fb4_to_mxfp8 applied to the output
 * of fb4_quantize_affine, byte for byte.  Default configuration and C a multiple of 64 only, gain and
 * bias 16-byte aligned (FB4_ERR_INVALID_ARG / FB4_ERR_SHAPE / FB4_ERR_ALIGN otherwise).
 *   e4m3, scales, scale_layout : as in fb4_quantize_mxfp8
 */
int fb4_quantize_affine_mxfp8(fb4_ctx* ctx, const void* x_bf16, int64_t T, int64_t C, int64_t ld_elems,
                              const void* gain_bf16, const void* bias_bf16, int gain_plus_one,
                              const int32_t* cluster_id, const uint32_t* cluster_mask, int32_t n_clusters,
                              uint8_t* e4m3, uint8_t* scales, int scale_layout, void* stream);

/*
 * LayerNorm with per-channel modulation fused in front of the quantizer (App. D.2 lists LayerNorm among the
 * operations the quantizer runs behind; in the adaLN blocks the normalised activation is modulated as
 * y = n * (1 + scale_c) + shift_c before the linear layer).  Per token, in float32:
 *     mean = sum(x) / C,  d = x - mean,  var = sum(d * d) / C,  rstd = 1 / sqrt(var + eps),
 *     y[c] = (d[c] * rstd) * g_c + bias_c,   g_c = gain_c (gain_plus_one 0) or 1 + gain_c (1),
 * every operation rounded once (IEEE binary32, nearest even; square root and divisions correctly rounded),
 * d * d + q and (d * rstd) * g + bias as fused multiply-adds, and the additions in a fixed order: the
 * 32 channels of a block in index order; the 32 block sums of a run of 1024 channels by an xor butterfly
 * (v_i <- v_i + v_(i xor off) for off = 16, 8, 4, 2, 1, all i at once; the run's sum is v_0); the runs of a
 * token added to +0 in order.  The result is therefore reproducible bit for bit; it is quantized from registers as
 * fb4_quantize_f32 quantizes a float32 tensor, so the token is read once and y never exists in memory.
 * Optional SeDA restriction as in fb4_quantize_seda.  One fused pass; default configuration only,
 * contiguous rows (ld_elems == C), C a multiple of 1024 and at most 16384, gain and bias 16-byte
 * aligned: FB4_ERR_INVALID_ARG for another configuration, FB4_ERR_SHAPE for another shape.
 *   x    : device bfloat16 [T][C]
 *   gain : device bfloat16 [C];  bias : device bfloat16 [C]
 *   eps  : added to the variance (>= 0, finite)
 */
int fb4_quantize_layernorm(fb4_ctx* ctx, const void* x_bf16, int64_t T, int64_t C, int64_t ld_elems,
                           const void* gain_bf16, const void* bias_bf16, int gain_plus_one, float eps,
                           const int32_t* cluster_id, const uint32_t* cluster_mask, int32_t n_clusters,
                           uint8_t* codes, uint16_t* meta, void* stream);

/*
 * SeDA-constrained quantization (Sec. 3.4): token t may only use the dialects in
 * cluster_mask[cluster_id[t]] (its cluster's sub-formatbook); cluster_id[t] == -1
 * means unconstrained.  Stage 1 is intersected with the mask; if the intersection
 * is empty the whole mask is scored.
 *   cluster_id   : device int32 [T], values in [-1, n_clusters).  The kernels check the range: any
 *                  other value is treated as -1 and raises bit 1 of the status word
 *                  (fb4_device_status); the mask table is never read out of bounds
 *   cluster_mask : device uint32 [n_clusters], every entry non-zero (precondition;
 *                  a zero mask yields dialect 0 for the affected tokens)
 */
int fb4_quantize_seda(fb4_ctx* ctx, const void* x_bf16, int64_t T, int64_t C, int64_t ld_elems,
                      const int32_t* cluster_id, const uint32_t* cluster_mask, int32_t n_clusters, uint8_t* codes,
                      uint16_t* meta, void* stream);

/*
 * Sub-formatbook construction for SeDA (Sec. 3.4: a per-cluster histogram of the dialects chosen
 * on the anchor tokens, of which every dynamic-range bucket keeps its most frequent member).
 * `meta` is the metadata of a quantization of
 * the layer's activation (normally unconstrained); anchor a is token anchor_token[a] and belongs
 * to cluster anchor_cluster[a].  For every cluster the dialect ids of all blocks of its anchor
 * tokens are counted; for every dynamic-range bucket (a distinct entry of the context's stage-1
 * table) the most frequent member is kept, ties and buckets without any count going to the
 * lowest dialect id.  cluster_mask[c] (the input of fb4_quantize_seda) = the kept dialects.
 *   meta           : device uint16 [T][C/B]
 *   anchor_token   : device int32 [n_anchor]; entries outside [0,T) are ignored
 *   anchor_cluster : device int32 [n_anchor]; entries outside [0,n_clusters) are ignored
 *   counts         : device uint32 [n_clusters][32], scratch provided by the caller; holds the
 *                    per-cluster dialect counts on return (n_anchor * C/B must stay below 2^32)
 *   cluster_mask   : device uint32 [n_clusters] (out)
 */
int fb4_build_subformatbook(fb4_ctx* ctx, const uint16_t* meta, int64_t T, int64_t C, const int32_t* anchor_token,
                            const int32_t* anchor_cluster, int64_t n_anchor, int32_t n_clusters, uint32_t* counts,
                            uint32_t* cluster_mask, void* stream);

/*
 * fb4_build_subformatbook without any device allocation (the paper has no counterpart; this is
 * a packaging of the call above).  It is meant for code that holds a context from start-up but
 * cannot obtain device memory at the point of the call: a plug-in that gets only the tensors
 * its host runtime hands it, a serving loop whose memory plan is frozen, a caller whose
 * allocator is off limits at that moment.  Such a caller has nowhere to get the `counts`
 * scratch from, so this variant keeps the counts in an array built into the library image.
 *   - Limit: n_clusters <= FB4_STATIC_MAX_CLUSTERS (1024); more returns FB4_ERR_STATIC_LIMIT and
 *     launches nothing.  The array (128 KB) occupies every GPU the library is loaded on until
 *     the process ends.
 *   - The call itself allocates nothing and frees nothing, on the device or through any
 *     library.  The first call on a device asks the CUDA runtime once for the array's address
 *     on that device; make that first call outside any stream capture.
 *   - All calls on a GPU share the one array, which still holds the previous call's counts:
 *     each call clears the part it uses (on `stream`) before counting.  Two calls that may run
 *     at the same time on one GPU (different streams, different contexts, different threads)
 *     race on it and give wrong masks; order them, or use fb4_build_subformatbook with
 *     separate scratch.
 *   - The context's device must be the current device.  Arguments, ignored anchors, tie rules
 *     and the result are those of fb4_build_subformatbook; the counts are not returned.
 */
#define FB4_STATIC_MAX_CLUSTERS 1024
int fb4_build_subformatbook_static(fb4_ctx* ctx, const uint16_t* meta, int64_t T, int64_t C,
                                   const int32_t* anchor_token, const int32_t* anchor_cluster, int64_t n_anchor,
                                   int32_t n_clusters, uint32_t* cluster_mask, void* stream);

/*
 * Salient-token selection for activation decomposition (Sec. 3.3: every tile of
 * tokens contributes its single highest-scoring token): for every tile of
 * `tile` consecutive tokens, the index of the largest score (ties: lowest index).
 *   score       : device float [T] (finite)
 *   salient_idx : device int32 [ceil(T/tile)], ascending on return
 */
int fb4_select_salient(fb4_ctx* ctx, const float* score, int64_t T, int32_t tile, int32_t* salient_idx,
                       void* stream);

/*
 * The global alternative to the per-tile selection: the k highest-scoring tokens of the whole
 * sequence, ties to the lowest index, written in ascending token order (the input format of
 * fb4_quantize_decomposed_idx).  Sec. 3.3 selects per tile and App. F argues against a global
 * top-k; this call exists for workloads stated as "the top p % of the tokens by score".
 * Sequences of 8192 to 16 Mi tokens run as a few small launches over many thread blocks (a radix
 * select with histograms in scratch memory of the context, then an ordered write); others as one
 * thread block.  Calls on one context must not overlap in time (different streams): they share
 * that scratch.
 *   score       : device float [T] (finite; -0 counts as +0)
 *   salient_idx : device int32 [k] (out), 0 <= k <= T
 */
int fb4_select_salient_topk(fb4_ctx* ctx, const float* score, int64_t T, int64_t k, int32_t* salient_idx,
                            void* stream);

/*
 * Quantization with activation decomposition (Sec. 3.3): every token is quantized
 * as in fb4_quantize[_seda]; for the salient tokens the residual
 * Delta = x - dequant(Q(x)) is formed in registers (exactly, in fp32), quantized
 * again with the same candidate set, and written compactly: row s of res_codes /
 * res_meta belongs to token salient_idx[s].  The salient set is selected first
 * from `score` (see fb4_select_salient) and returned in salient_idx.
 *   cluster_id   : NULL = no SeDA restriction (then cluster_mask is ignored)
 *   salient_idx  : device int32 [ceil(T/tile)] (out)
 *   res_codes    : device uint8  [ceil(T/tile)][C/2] (out)
 *   res_meta     : device uint16 [ceil(T/tile)][C/B] (out)
 */
int fb4_quantize_decomposed(fb4_ctx* ctx, const void* x_bf16, int64_t T, int64_t C, int64_t ld_elems,
                            const float* score, int32_t tile, const int32_t* cluster_id,
                            const uint32_t* cluster_mask, int32_t n_clusters, uint8_t* codes, uint16_t* meta,
                            int32_t* salient_idx, uint8_t* res_codes, uint16_t* res_meta, void* stream);

/*
 * The same with a salient set given by the caller (App. C: layers that precede the
 * attention computation reuse the previous timestep's salient tokens).
 *   salient_idx : device int32 [n_salient] (in), strictly ascending, each in [0,T)
 *                 (precondition; not checked on the device)
 */
int fb4_quantize_decomposed_idx(fb4_ctx* ctx, const void* x_bf16, int64_t T, int64_t C, int64_t ld_elems,
                                const int32_t* salient_idx, int64_t n_salient, const int32_t* cluster_id,
                                const uint32_t* cluster_mask, int32_t n_clusters, uint8_t* codes,
                                uint16_t* meta, uint8_t* res_codes, uint16_t* res_meta, void* stream);

/*
 * Decode (App. D.2: 4-bit codes are decoded on the fly with the block scale applied):
 * out[t][c] = value(codes, meta); for tokens listed in salient_idx the decoded
 * residual is added, the sum rounded once to fp32 (Sec. 3.3: Q(Act)+Q(Delta)).
 *   salient_idx : NULL / n_salient = 0 for plain tensors; else device int32
 *                 [n_salient], strictly ascending.  An entry outside [0, T) is skipped (its
 *                 residual row is not added anywhere) and raises bit 1 of the status word
 *   out         : device, [T][C] contiguous; out_dtype 0 = float32, 1 = bfloat16, 2 = IEEE half
 *                 (the type App. D.2 decodes to); 1 and 2 are the round-to-nearest-even of the
 *                 fp32 result (half: overflow to infinity, gradual underflow)
 */
int fb4_dequantize(fb4_ctx* ctx, const uint8_t* codes, const uint16_t* meta, int64_t T, int64_t C,
                   const int32_t* salient_idx, int64_t n_salient, const uint8_t* res_codes,
                   const uint16_t* res_meta, void* out, int out_dtype, void* stream);

/*
 * Offline weight quantization (Sec. 3.3: weights are known ahead of time, so their dialects can be
 * searched exhaustively with no approximation; App. C: the criterion is the squared error).  Same
 * format and scale as fb4_quantize, but the dialect of a block is the one with the smallest
 * squared error over ALL its elements among ALL 32 dialects (no groups, no stage 1, no error
 * table), ties to the lowest id.  The errors are summed in double precision in element order.
 * Uses the context's block size and exponent clamp.  Not a bandwidth path.
 *   w : device bfloat16 [N][ld_elems]; blocks run along the K (contiguous) axis
 */
int fb4_quantize_weights(fb4_ctx* ctx, const void* w_bf16, int64_t N, int64_t K, int64_t ld_elems, uint8_t* codes,
                         uint16_t* meta, void* stream);

/*
 * MXFP8 view of a quantized tensor (App. D.2: every integer magnitude 0..15 is an e4m3 number and
 * the block scale is a power of two, so an FB4 tensor is an MXFP8 GEMM operand as it stands).
 * Element -> the e4m3 byte of its signed magnitude; block -> the E8M0 byte of its
 * element scale 2^(e-3), which is the scale byte of `meta`.  Exact: e4m3 * scale equals the value
 * fb4_dequantize gives.  Block size 32 only (FB4_ERR_INVALID_ARG otherwise); residual tensors
 * (res_codes / res_meta) are converted by a second call.
 *   e4m3         : device uint8 [T][C] (out), 16-byte aligned
 *   scales       : device uint8 (out), fb4_mxfp8_scale_bytes(T, C, scale_layout) bytes
 *   scale_layout : 0 = row-major [T][C/32];
 *                  1 = tiles of 128 rows x 4 scale columns (512 bytes each; the column tiles of a
 *                      band of 128 rows follow one another), scale (r, c) of a tile at byte
 *                      (r mod 32)*16 + (r div 32)*4 + c: the order block-scaled tensor-core GEMMs
 *                      read scale factors in.  Rows are padded to a multiple of 128 and scale
 *                      columns to a multiple of 4; padding bytes are written as 0x7f (scale 1).
 */
int fb4_to_mxfp8(fb4_ctx* ctx, const uint8_t* codes, const uint16_t* meta, int64_t T, int64_t C, uint8_t* e4m3,
                 uint8_t* scales, int scale_layout, void* stream);
/*
 * fb4_quantize[_seda] and fb4_to_mxfp8 in one pass (App. D.2 names an MXFP8 GEMM on Blackwell as
 * the consumer of FB4): x is quantized as in fb4_quantize / fb4_quantize_seda, and the result is
 * written directly as e4m3 bytes and E8M0 scales; the 4-bit codes and the dialect ids are not
 * stored (3.03 instead of 2.56 + 1.59 bytes per element of traffic).  The output equals
 * fb4_to_mxfp8 applied to the output of fb4_quantize[_seda], byte for byte.
 * Default configuration only (block size 32, num_groups 8, two-stage selection, full exponent
 * range, a formatbook that fits the packed tables) and C a multiple of 64: otherwise
 * FB4_ERR_INVALID_ARG / FB4_ERR_SHAPE, and the two calls are used instead.
 *   cluster_id : NULL = no SeDA restriction (then cluster_mask is ignored)
 *   e4m3       : device uint8 [T][C] (out), 32-byte aligned
 *   scales     : device uint8 (out), fb4_mxfp8_scale_bytes(T, C, scale_layout) bytes; with the
 *                tiled layout and T or C/32 not a multiple of 128 / 4 the whole buffer is first
 *                filled with 0x7f (scale 1) on the stream
 */
int fb4_quantize_mxfp8(fb4_ctx* ctx, const void* x_bf16, int64_t T, int64_t C, int64_t ld_elems,
                       const int32_t* cluster_id, const uint32_t* cluster_mask, int32_t n_clusters, uint8_t* e4m3,
                       uint8_t* scales, int scale_layout, void* stream);

/*
 * fb4_quantize_mxfp8 with activation decomposition (Sec. 3.3: Act ~ Q(Act) + Q(Delta) for salient
 * tokens; App. D.2: the consumer is an MXFP8 GEMM): one pass writes Q(Act) as an MXFP8 operand
 * [T][C] and Q(Delta) of the salient tokens as a second, compact MXFP8 operand [n_salient][C].
 * The sum of the two is not an e4m3 value in general, so the residual stays a separate operand:
 * the consumer multiplies it as a second, small GEMM and adds the rows listed in salient_idx.
 * The outputs equal fb4_to_mxfp8 applied to the main and to the residual output of
 * fb4_quantize_decomposed[_idx], byte for byte.  Same restrictions as fb4_quantize_mxfp8.
 *   score        : device float [T] -> one salient token per `tile` tokens is selected first
 *                  (fb4_select_salient) and written to salient_idx (capacity ceil(T/tile));
 *                  NULL -> salient_idx is an input: n_salient strictly ascending token ids
 *   n_salient    : used only when score is NULL
 *   cluster_id   : NULL = no SeDA restriction; else main and residual both use the token's mask
 *   res_e4m3     : device uint8 [n_salient][C] (out), 32-byte aligned
 *   res_scales   : device uint8 (out), fb4_mxfp8_scale_bytes(n_salient, C, scale_layout) bytes,
 *                  the scale layout applied to the residual operand on its own
 */
int fb4_quantize_mxfp8_decomposed(fb4_ctx* ctx, const void* x_bf16, int64_t T, int64_t C, int64_t ld_elems,
                                  const float* score, int32_t tile, int32_t* salient_idx, int64_t n_salient,
                                  const int32_t* cluster_id, const uint32_t* cluster_mask, int32_t n_clusters,
                                  uint8_t* e4m3, uint8_t* scales, uint8_t* res_e4m3, uint8_t* res_scales,
                                  int scale_layout, void* stream);

/* Size in bytes of the scale buffer of fb4_to_mxfp8 (-1 for invalid arguments).  Host only. */
int64_t fb4_mxfp8_scale_bytes(int64_t T, int64_t C, int scale_layout);

/*
 * Host-buffer form of fb4_quantize for callers whose tensors live in host memory:
 * copies x from the host, quantizes, and copies codes and meta back, in row
 * chunks pipelined over the context's own streams, then waits for completion.
 *   x_host, codes_host, meta_host : HOST pointers (pinned memory overlaps copies
 *                                   with compute; pageable memory works, slower)
 *   d_x, d_codes, d_meta          : DEVICE staging buffers of the full tensor
 *                                   sizes, provided by the caller
 */
int fb4_quantize_host(fb4_ctx* ctx, const void* x_host, int64_t T, int64_t C, void* d_x, uint8_t* d_codes,
                      uint16_t* d_meta, uint8_t* codes_host, uint16_t* meta_host);

/* Kernel choice: 0 (default) = the TMA-staged kernel whenever the call qualifies (num_groups 8,
 * two-stage selection, a formatbook whose stage-1 groups hold at most 8 dialects, C a multiple
 * of 64; either block size, any exponent clamp, every extension), else the generic kernel;
 * 1 = always the generic kernel (and the single-block form of fb4_select_salient_topk).  Both
 * choices produce identical output; this exists for tests and measurements. */
int fb4_set_kernel_variant(fb4_ctx* ctx, int variant);

/* Device-side status word of the context, read back with a blocking copy: 0 = fine; bit 0 =
 * a bounded wait on an asynchronous (TMA) load inside a kernel ran out of tries, in which case
 * the affected warp stopped early and the outputs of that call are incomplete; bit 1 = an index
 * argument on the device (a cluster id, a salient token index on decode) was outside its table
 * and was handled as documented at the call.  Bits stay set for the life of the context. */
int fb4_device_status(fb4_ctx* ctx, uint32_t* status);

/* Number of kernel launches this context has enqueued so far (diagnostic counter). */
int64_t fb4_launch_count(const fb4_ctx* ctx);

/* Name of the kernel variant the last quantize call on this context used
 * ("fast" = TMA-staged sm_100a path, "generic" = fallback for other shapes). */
const char* fb4_last_variant(const fb4_ctx* ctx);

/* cudaError_t of the last failing CUDA call made through this library (0 if none). */
int fb4_last_cuda_error(void);

const char* fb4_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* FB4_H_ */
