// Internal declarations shared by the translation units of libfb4 (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "fb4.h"

// Lookup tables as they sit in device global memory (copied to shared memory by each CTA).
struct Fb4DeviceTables {
  uint8_t qvalue[32][32];   // [dialect][bin] -> index 0..7 of the nearest magnitude   (Sec. 3.2)
  uint8_t qerror[32][32];   // [dialect][bin] -> |bin midpoint - nearest magnitude| in quarter units
  uint8_t formatbook[32][8];
  uint32_t stage1[32];      // [bin of block maximum] -> candidate dialect mask
};

// Stage-1 table passed to a kernel by value.
struct Fb4Stage1 {
  uint32_t m[32];
};

// Per-row extras of one quantize launch (all pointers device, nullable).
struct Fb4RowExtras {
  const int32_t* cluster_id;    // SeDA: token -> cluster, -1 = unconstrained
  const uint32_t* cluster_mask; // SeDA: cluster -> allowed dialect mask
  int32_t n_clusters;           // entries of cluster_mask; ids outside [-1, n_clusters) count as -1 and raise status bit 1
  const int32_t* salient_idx;   // ascending token ids whose residual is quantized too
  int64_t n_salient;
  int32_t tile;                 // > 0: salient_idx[t / tile] is the only possible match for token t
  uint8_t* res_codes;           // [n_salient][C/2]
  uint16_t* res_meta;           // [n_salient][C/B]
};

// The tensor map of the last launch of each kernel family (encoding one costs a good part of a microsecond on the
// host; a layer quantizes the same buffer step after step).
struct Fb4TensorMapSlot {
  const void* x;
  int64_t T, C, ld;
  int valid;
  alignas(64) unsigned char map[128];
};

struct fb4_ctx {
  int device;
  mutable Fb4TensorMapSlot tmap_slot[4];   // 0: strided bf16, 1: flat, 2 KB tiles, 2: flat, 4 KB tiles, 3: fp32 input
  fb4_config cfg;
  Fb4DeviceTables host_tables;   // host copy
  Fb4DeviceTables* d_tables;     // device copy
  void* d_fast_tables;           // packed tables of the TMA-staged kernel (NULL if not eligible)
  size_t fast_table_bytes;
  int force_generic;             // fb4_set_kernel_variant(ctx, 1): always take the generic kernel
  int fast_ok;                   // formatbook/stage-1 table fit the fast kernel's packed layout
  int sm_count;
  void* d_topk_scratch;          // histograms and counters of the multi-CTA top-k selection (fb4_topk.cu)
  uint32_t* d_status;            // device status word (bit 0: a TMA wait ran out of tries; bit 1: an index argument out of range)
  int64_t launches;
  const char* last_variant;
  cudaStream_t pipe_stream[3];   // fb4_quantize_host pipeline
  cudaEvent_t pipe_event[3];
};

int fb4_set_cuda_error(cudaError_t e);   // records e, returns FB4_ERR_CUDA

// TMA-staged kernel of the default configuration (fb4_fast.cu)
bool fb4_fast_build_tables(const Fb4DeviceTables& t, int select_mode, void** d_out, size_t* bytes);
cudaError_t fb4_fast_prepare_device();
bool fb4_fast_eligible(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld);
cudaError_t fb4_launch_quantize_fast(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld,
                                     const Fb4RowExtras& ex, uint8_t* codes, uint16_t* meta, cudaStream_t stream);

bool fb4_fast_mx_eligible(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld);
cudaError_t fb4_launch_quantize_fast_mx(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld,
                                        const Fb4RowExtras& ex, uint8_t* e4m3, uint8_t* scales, uint8_t* res_e4m3,
                                        uint8_t* res_scales, int tiled, cudaStream_t stream, int* launches);
bool fb4_fast_affine_eligible(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, const void* gain,
                              const void* bias);
cudaError_t fb4_launch_quantize_fast_affine(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld,
                                            const void* gain, const void* bias, int plus_one,
                                            const Fb4RowExtras& ex, uint8_t* codes, uint16_t* meta,
                                            cudaStream_t stream, uint8_t* e4m3 = nullptr, uint8_t* scales = nullptr,
                                            int tiled = 0);   // e4m3 != NULL: MXFP8 output instead of codes / meta
bool fb4_fast_layernorm_eligible(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, const void* gain,
                                 const void* bias);
cudaError_t fb4_launch_quantize_layernorm(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, const void* gain,
                                          const void* bias, int plus_one, float eps, const Fb4RowExtras& ex,
                                          uint8_t* codes, uint16_t* meta, cudaStream_t stream);
bool fb4_fast_f32_eligible(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld);
cudaError_t fb4_launch_quantize_fast_f32(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld,
                                         uint8_t* codes, uint16_t* meta, cudaStream_t stream);

// generic kernels (any supported config)
cudaError_t fb4_launch_quantize_generic(const fb4_ctx* ctx, const void* x, int x_is_f32, int64_t T, int64_t C,
                                        int64_t ld, const Fb4RowExtras& ex, uint8_t* codes, uint16_t* meta,
                                        cudaStream_t stream, const void* gain = nullptr, const void* bias = nullptr,
                                        int plus_one = 0);   // gain/bias: affine producer in front (bf16 input only)
cudaError_t fb4_launch_dequantize(const fb4_ctx* ctx, const uint8_t* codes, const uint16_t* meta, int64_t T,
                                  int64_t C, const int32_t* salient_idx, int64_t n_salient,
                                  const uint8_t* res_codes, const uint16_t* res_meta, void* out, int out_dtype,
                                  cudaStream_t stream, int* launches);
cudaError_t fb4_launch_subformatbook(const uint16_t* meta, int64_t T, int64_t nblk, const int32_t* anchor_token,
                                     const int32_t* anchor_cluster, int64_t n_anchor, int32_t n_clusters,
                                     const Fb4Stage1& stage1, uint32_t* counts, uint32_t* cluster_mask, int sm_count,
                                     cudaStream_t stream, int* launches);
cudaError_t fb4_launch_quantize_weights(const fb4_ctx* ctx, const void* w, int64_t N, int64_t K, int64_t ld,
                                        uint8_t* codes, uint16_t* meta, cudaStream_t stream);
cudaError_t fb4_launch_to_mxfp8(const fb4_ctx* ctx, const uint8_t* codes, const uint16_t* meta, int64_t T, int64_t C,
                                uint8_t* e4m3, uint8_t* scales, int layout, cudaStream_t stream);
size_t fb4_topk_scratch_bytes();
bool fb4_topk_multi_eligible(int64_t T);
cudaError_t fb4_launch_select_salient_topk_multi(const fb4_ctx* ctx, const float* score, int64_t T, int64_t k,
                                                 int32_t* salient_idx, cudaStream_t stream, int* launches);
cudaError_t fb4_launch_select_salient_topk(const float* score, int64_t T, int64_t k, int32_t* salient_idx,
                                           cudaStream_t stream);
cudaError_t fb4_launch_select_salient(const float* score, int64_t T, int32_t tile, int32_t* salient_idx,
                                      cudaStream_t stream);
