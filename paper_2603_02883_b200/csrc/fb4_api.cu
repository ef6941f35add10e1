// C-ABI entry points of libfb4: argument checks, context and lookup-table construction,
// kernel dispatch.  See include/fb4.h for the contract of every call.
#include <atomic>
#include <cstring>
#include <new>

#include "fb4_internal.h"

namespace {

std::atomic<int> g_last_cuda_error{0};

// Built-in stand-in formatbook (the paper's own table is only shown in Fig. 2a): designed from the
// four rules of Sec. 3.1; dialects per dynamic range 8..15 = 2,2,3,3,4,5,6,7; ids ascend with range.
const uint8_t kStandinFormatbook[32][8] = {
    {0, 1, 2, 3, 4, 5, 6, 8},    {0, 1, 2, 4, 5, 6, 7, 8},
    {0, 1, 2, 3, 4, 5, 7, 9},    {0, 1, 2, 4, 6, 7, 8, 9},
    {0, 1, 2, 3, 4, 6, 8, 10},   {0, 1, 2, 3, 5, 7, 9, 10},   {0, 1, 2, 4, 6, 8, 9, 10},
    {0, 1, 2, 3, 4, 6, 8, 11},   {0, 1, 2, 3, 5, 7, 9, 11},   {0, 1, 2, 4, 6, 8, 10, 11},
    {0, 1, 2, 3, 4, 6, 8, 12},   {0, 1, 2, 3, 5, 7, 9, 12},   {0, 1, 2, 4, 6, 8, 10, 12},
    {0, 2, 4, 6, 8, 10, 11, 12},
    {0, 1, 2, 3, 4, 6, 9, 13},   {0, 1, 2, 3, 5, 7, 10, 13},  {0, 1, 2, 4, 6, 8, 10, 13},
    {0, 1, 2, 4, 6, 9, 11, 13},  {0, 2, 4, 6, 8, 10, 12, 13},
    {0, 1, 2, 3, 4, 6, 9, 14},   {0, 1, 2, 3, 5, 7, 10, 14},  {0, 1, 2, 4, 6, 8, 11, 14},
    {0, 1, 2, 4, 6, 9, 12, 14},  {0, 1, 3, 5, 7, 9, 12, 14},  {0, 2, 4, 6, 8, 10, 12, 14},
    {0, 1, 2, 3, 4, 6, 9, 15},   {0, 1, 2, 3, 5, 7, 10, 15},  {0, 1, 2, 4, 6, 8, 11, 15},
    {0, 1, 2, 4, 6, 9, 12, 15},  {0, 1, 3, 5, 7, 9, 12, 15},  {0, 1, 3, 5, 7, 10, 13, 15},
    {0, 2, 4, 6, 8, 11, 13, 15},
};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool config_valid(const fb4_config& c) {
  if (c.block_size != 32 && c.block_size != 16) return false;
  if (c.num_groups != 8 && c.num_groups != c.block_size) return false;
  if (c.exp_min < -124 || c.exp_max > 127 || c.exp_min > c.exp_max) return false;
  if (c.select_mode > 1) return false;
  return true;
}

// Sec. 3.2 lookup tables.  Magnitudes are integers, so the decision boundary between two
// neighbouring magnitudes a < b is (a+b)/2, i.e. bin a+b in units of 0.5: every bin lies
// entirely on one side of every boundary, which makes Qvalue exact.
void build_tables(Fb4DeviceTables& t, const uint8_t* fb, const uint32_t* stage1) {
  std::memcpy(t.formatbook, fb, 256);
  for (int d = 0; d < 32; ++d) {
    for (int k = 0; k < 32; ++k) {
      int idx = 0;
      for (int j = 1; j < 8; ++j)
        if ((int)t.formatbook[d][j - 1] + (int)t.formatbook[d][j] <= k) idx = j;
      t.qvalue[d][k] = (uint8_t)idx;
      const int q = 2 * k + 1 - 4 * (int)t.formatbook[d][idx];   // midpoint k/2+1/4, quarter units
      t.qerror[d][k] = (uint8_t)(q < 0 ? -q : q);
    }
  }
  for (int k = 0; k < 32; ++k) {
    if (stage1) {
      t.stage1[k] = stage1[k];
    } else {
      const int bucket = (k >> 1) < 8 ? 8 : (k >> 1);
      uint32_t m = 0;
      for (int d = 0; d < 32; ++d)
        if (t.formatbook[d][7] == bucket) m |= 1u << d;
      t.stage1[k] = m;
    }
  }
}

int check_quantize_args(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, const void* codes,
                        const void* meta) {
  if (!ctx) return FB4_ERR_INVALID_ARG;
  if (T < 0 || C <= 0 || C % ctx->cfg.block_size != 0 || ld < C) return FB4_ERR_SHAPE;
  if (T == 0) return FB4_OK;
  if (!x || !codes || !meta) return FB4_ERR_INVALID_ARG;
  if (T > 0x7fffffffLL) return FB4_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(codes) || !aligned16(meta) || (ld & 7)) return FB4_ERR_ALIGN;
  return FB4_OK;
}

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

int run_quantize(fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, const Fb4RowExtras& ex,
                 uint8_t* codes, uint16_t* meta, cudaStream_t stream) {
  if (T == 0) return FB4_OK;
  cudaError_t e;
  if (!ctx->force_generic && fb4_fast_eligible(ctx, x, T, C, ld)) {
    e = fb4_launch_quantize_fast(ctx, x, T, C, ld, ex, codes, meta, stream);
    ctx->last_variant = "fast";
  } else {
    e = fb4_launch_quantize_generic(ctx, x, 0, T, C, ld, ex, codes, meta, stream);
    ctx->last_variant = "generic";
  }
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  ctx->launches += 1;
  return FB4_OK;
}

}  // namespace

int fb4_set_cuda_error(cudaError_t e) {
  g_last_cuda_error.store((int)e);
  return FB4_ERR_CUDA;
}

extern "C" {

void fb4_default_config(fb4_config* cfg) {
  if (!cfg) return;
  cfg->block_size = 32;
  cfg->num_groups = 8;
  cfg->exp_min = -124;
  cfg->exp_max = 127;
  cfg->select_mode = 0;
}

int fb4_init(fb4_ctx** out, int device, const uint8_t* formatbook, const uint32_t* stage1_mask,
             const fb4_config* cfg) {
  if (!out) return FB4_ERR_INVALID_ARG;
  *out = nullptr;
  fb4_config c;
  fb4_default_config(&c);
  if (cfg) c = *cfg;
  if (!config_valid(c)) return FB4_ERR_INVALID_ARG;
  const uint8_t* fb = formatbook ? formatbook : &kStandinFormatbook[0][0];
  for (int d = 0; d < 32; ++d) {
    if (fb[d * 8] != 0) return FB4_ERR_FORMATBOOK;
    for (int j = 1; j < 8; ++j)
      if (fb[d * 8 + j] <= fb[d * 8 + j - 1] || fb[d * 8 + j] > 15) return FB4_ERR_FORMATBOOK;
  }
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) {
    cudaGetLastError();
    return FB4_ERR_NO_DEVICE;
  }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return fb4_set_cuda_error(cudaGetLastError());
  if (prop.major != 10) return FB4_ERR_NO_DEVICE;   // kernels are built for sm_100a only

  fb4_ctx* ctx = new (std::nothrow) fb4_ctx();
  if (!ctx) return FB4_ERR_INVALID_ARG;
  ctx->device = device;
  ctx->cfg = c;
  ctx->sm_count = prop.multiProcessorCount;
  ctx->launches = 0;
  ctx->last_variant = "none";
  ctx->d_tables = nullptr;
  ctx->d_fast_tables = nullptr;
  ctx->fast_ok = 0;
  ctx->force_generic = 0;
  ctx->d_status = nullptr;
  ctx->d_topk_scratch = nullptr;
  for (int i = 0; i < 3; ++i) { ctx->pipe_stream[i] = nullptr; ctx->pipe_event[i] = nullptr; }
  build_tables(ctx->host_tables, fb, stage1_mask);

  DeviceGuard guard(device);
  if (!guard.ok) { delete ctx; return fb4_set_cuda_error(cudaGetLastError()); }
  cudaError_t e = cudaMalloc(&ctx->d_tables, sizeof(Fb4DeviceTables));
  if (e == cudaSuccess)
    e = cudaMemcpy(ctx->d_tables, &ctx->host_tables, sizeof(Fb4DeviceTables), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->d_status, sizeof(uint32_t));
  if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, sizeof(uint32_t));
  if (e == cudaSuccess) e = cudaMalloc(&ctx->d_topk_scratch, fb4_topk_scratch_bytes());
  if (e != cudaSuccess) {
    if (ctx->d_topk_scratch) cudaFree(ctx->d_topk_scratch);
    if (ctx->d_status) cudaFree(ctx->d_status);
    if (ctx->d_tables) cudaFree(ctx->d_tables);
    delete ctx;
    return fb4_set_cuda_error(e);
  }
  size_t fast_bytes = 0;
  if (fb4_fast_build_tables(ctx->host_tables, c.select_mode, &ctx->d_fast_tables, &fast_bytes) &&
      fb4_fast_prepare_device() == cudaSuccess)
    ctx->fast_ok = 1;
  ctx->fast_table_bytes = fast_bytes;
  cudaGetLastError();
  *out = ctx;
  return FB4_OK;
}

int fb4_destroy(fb4_ctx* ctx) {
  if (!ctx) return FB4_OK;
  DeviceGuard guard(ctx->device);
  for (int i = 0; i < 3; ++i) {
    if (ctx->pipe_event[i]) cudaEventDestroy(ctx->pipe_event[i]);
    if (ctx->pipe_stream[i]) cudaStreamDestroy(ctx->pipe_stream[i]);
  }
  if (ctx->d_fast_tables) cudaFree(ctx->d_fast_tables);
  if (ctx->d_topk_scratch) cudaFree(ctx->d_topk_scratch);
  if (ctx->d_status) cudaFree(ctx->d_status);
  if (ctx->d_tables) cudaFree(ctx->d_tables);
  delete ctx;
  return FB4_OK;
}

int fb4_block_tables(const fb4_ctx* ctx, const void** device_image, uint64_t* bytes) {
  if (!ctx || !device_image || !bytes) return FB4_ERR_INVALID_ARG;
  const fb4_config& c = ctx->cfg;
  if (!ctx->fast_ok || !ctx->d_fast_tables || c.block_size != 32 || c.num_groups != 8 || c.select_mode != 0 ||
      c.exp_min != -124 || c.exp_max != 127)
    return FB4_ERR_INVALID_ARG;
  *device_image = ctx->d_fast_tables;
  *bytes = ctx->fast_table_bytes;
  return FB4_OK;
}

int fb4_get_tables(const fb4_ctx* ctx, uint8_t* formatbook, uint32_t* stage1_mask, uint8_t* qvalue,
                   uint8_t* qerror_q4) {
  if (!ctx) return FB4_ERR_INVALID_ARG;
  if (formatbook) std::memcpy(formatbook, ctx->host_tables.formatbook, 256);
  if (stage1_mask) std::memcpy(stage1_mask, ctx->host_tables.stage1, 128);
  if (qvalue) std::memcpy(qvalue, ctx->host_tables.qvalue, 1024);
  if (qerror_q4) std::memcpy(qerror_q4, ctx->host_tables.qerror, 1024);
  return FB4_OK;
}

int fb4_quantize(fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, uint8_t* codes, uint16_t* meta,
                 void* stream) {
  const int rc = check_quantize_args(ctx, x, T, C, ld, codes, meta);
  if (rc != FB4_OK) return rc;
  Fb4RowExtras ex{};
  return run_quantize(ctx, x, T, C, ld, ex, codes, meta, static_cast<cudaStream_t>(stream));
}

int fb4_quantize_f32(fb4_ctx* ctx, const float* x, int64_t T, int64_t C, int64_t ld, uint8_t* codes, uint16_t* meta,
                     void* stream) {
  if (!ctx) return FB4_ERR_INVALID_ARG;
  if (T < 0 || C <= 0 || C % ctx->cfg.block_size != 0 || ld < C) return FB4_ERR_SHAPE;
  if (T == 0) return FB4_OK;
  if (!x || !codes || !meta) return FB4_ERR_INVALID_ARG;
  if (T > 0x7fffffffLL) return FB4_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(codes) || !aligned16(meta) || (ld & 3)) return FB4_ERR_ALIGN;
  cudaError_t e;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!ctx->force_generic && fb4_fast_f32_eligible(ctx, x, T, C, ld)) {
    e = fb4_launch_quantize_fast_f32(ctx, x, T, C, ld, codes, meta, st);
    ctx->last_variant = "fast";
  } else {
    Fb4RowExtras ex{};
    e = fb4_launch_quantize_generic(ctx, x, 1, T, C, ld, ex, codes, meta, st);
    ctx->last_variant = "generic";
  }
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  ctx->launches += 1;
  return FB4_OK;
}

int fb4_quantize_layernorm(fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, const void* gain,
                           const void* bias, int gain_plus_one, float eps, const int32_t* cluster_id,
                           const uint32_t* cluster_mask, int32_t n_clusters, uint8_t* codes, uint16_t* meta,
                           void* stream) {
  const int rc = check_quantize_args(ctx, x, T, C, ld, codes, meta);
  if (rc != FB4_OK) return rc;
  if (gain_plus_one != 0 && gain_plus_one != 1) return FB4_ERR_INVALID_ARG;
  if (!(eps >= 0.0f) || eps > 3.0e38f) return FB4_ERR_INVALID_ARG;
  const fb4_config& c = ctx->cfg;
  if (c.block_size != 32 || c.num_groups != 8 || c.select_mode != 0 || c.exp_min != -124 || c.exp_max != 127 ||
      !ctx->fast_ok)
    return FB4_ERR_INVALID_ARG;
  if (ld != C || C % 1024 != 0 || C > 16384 || T > 0x7fffffffLL) return FB4_ERR_SHAPE;
  if (T == 0) return FB4_OK;
  if (!gain || !bias) return FB4_ERR_INVALID_ARG;
  if (cluster_id && (!cluster_mask || n_clusters <= 0)) return FB4_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(gain) & 15u) || (reinterpret_cast<uintptr_t>(bias) & 15u)) return FB4_ERR_ALIGN;
  Fb4RowExtras ex{};
  ex.cluster_id = cluster_id;
  ex.cluster_mask = cluster_id ? cluster_mask : nullptr;
  ex.n_clusters = cluster_id ? n_clusters : 0;
  if (!fb4_fast_layernorm_eligible(ctx, x, T, C, ld, gain, bias)) return FB4_ERR_SHAPE;
  const cudaError_t e = fb4_launch_quantize_layernorm(ctx, x, T, C, gain, bias, gain_plus_one, eps, ex, codes, meta,
                                                      static_cast<cudaStream_t>(stream));
  ctx->last_variant = "fast";
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  ctx->launches += 1;
  return FB4_OK;
}

int fb4_quantize_affine(fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, const void* gain,
                        const void* bias, int gain_plus_one, const int32_t* cluster_id, const uint32_t* cluster_mask,
                        int32_t n_clusters, uint8_t* codes, uint16_t* meta, void* stream) {
  const int rc = check_quantize_args(ctx, x, T, C, ld, codes, meta);
  if (rc != FB4_OK) return rc;
  if (gain_plus_one != 0 && gain_plus_one != 1) return FB4_ERR_INVALID_ARG;
  if (T == 0) return FB4_OK;
  if (!gain || !bias) return FB4_ERR_INVALID_ARG;
  if (cluster_id && (!cluster_mask || n_clusters <= 0)) return FB4_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(gain) & 1u) || (reinterpret_cast<uintptr_t>(bias) & 1u)) return FB4_ERR_ALIGN;
  cudaError_t e;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  Fb4RowExtras ex{};
  ex.cluster_id = cluster_id;
  ex.cluster_mask = cluster_id ? cluster_mask : nullptr;
  ex.n_clusters = cluster_id ? n_clusters : 0;
  if (!ctx->force_generic && fb4_fast_affine_eligible(ctx, x, T, C, ld, gain, bias)) {
    e = fb4_launch_quantize_fast_affine(ctx, x, T, C, ld, gain, bias, gain_plus_one, ex, codes, meta, st);
    ctx->last_variant = "fast";
  } else {
    e = fb4_launch_quantize_generic(ctx, x, 0, T, C, ld, ex, codes, meta, st, gain, bias, gain_plus_one);
    ctx->last_variant = "generic";
  }
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  ctx->launches += 1;
  return FB4_OK;
}

int fb4_quantize_affine_mxfp8(fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, const void* gain,
                              const void* bias, int gain_plus_one, const int32_t* cluster_id,
                              const uint32_t* cluster_mask, int32_t n_clusters, uint8_t* e4m3, uint8_t* scales,
                              int scale_layout, void* stream) {
  if (!ctx) return FB4_ERR_INVALID_ARG;
  if (scale_layout != 0 && scale_layout != 1) return FB4_ERR_INVALID_ARG;
  if (gain_plus_one != 0 && gain_plus_one != 1) return FB4_ERR_INVALID_ARG;
  if (T < 0 || C <= 0 || C % 64 != 0 || ld < C || T > 0x7fffffffLL) return FB4_ERR_SHAPE;
  if (T == 0) return FB4_OK;
  if (!x || !gain || !bias || !e4m3 || !scales) return FB4_ERR_INVALID_ARG;
  if (cluster_id && (!cluster_mask || n_clusters <= 0)) return FB4_ERR_INVALID_ARG;
  if (!aligned16(x) || (ld & 7) || (reinterpret_cast<uintptr_t>(e4m3) & 31u) || !aligned16(gain) || !aligned16(bias))
    return FB4_ERR_ALIGN;
  if (!fb4_fast_affine_eligible(ctx, x, T, C, ld, gain, bias)) return FB4_ERR_INVALID_ARG;   // default configuration only
  Fb4RowExtras ex{};
  ex.cluster_id = cluster_id;
  ex.cluster_mask = cluster_id ? cluster_mask : nullptr;
  ex.n_clusters = cluster_id ? n_clusters : 0;
  const cudaError_t e = fb4_launch_quantize_fast_affine(ctx, x, T, C, ld, gain, bias, gain_plus_one, ex, nullptr,
                                                        nullptr, static_cast<cudaStream_t>(stream), e4m3, scales,
                                                        scale_layout);
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  ctx->launches += 1;
  ctx->last_variant = "fast";
  return FB4_OK;
}

int fb4_quantize_seda(fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, const int32_t* cluster_id,
                      const uint32_t* cluster_mask, int32_t n_clusters, uint8_t* codes, uint16_t* meta,
                      void* stream) {
  const int rc = check_quantize_args(ctx, x, T, C, ld, codes, meta);
  if (rc != FB4_OK) return rc;
  if (T > 0 && (!cluster_id || !cluster_mask || n_clusters <= 0)) return FB4_ERR_INVALID_ARG;
  Fb4RowExtras ex{};
  ex.cluster_id = cluster_id;
  ex.cluster_mask = cluster_mask;
  ex.n_clusters = n_clusters;
  return run_quantize(ctx, x, T, C, ld, ex, codes, meta, static_cast<cudaStream_t>(stream));
}

int fb4_select_salient(fb4_ctx* ctx, const float* score, int64_t T, int32_t tile, int32_t* salient_idx,
                       void* stream) {
  if (!ctx || tile <= 0) return FB4_ERR_INVALID_ARG;
  if (T < 0 || T > 0x7fffffffLL) return FB4_ERR_SHAPE;
  if (T == 0) return FB4_OK;
  if (!score || !salient_idx) return FB4_ERR_INVALID_ARG;
  cudaError_t e = fb4_launch_select_salient(score, T, tile, salient_idx, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  ctx->launches += 1;
  return FB4_OK;
}

int fb4_select_salient_topk(fb4_ctx* ctx, const float* score, int64_t T, int64_t k, int32_t* salient_idx,
                            void* stream) {
  if (!ctx) return FB4_ERR_INVALID_ARG;
  if (T < 0 || T > 0x7fffffffLL) return FB4_ERR_SHAPE;
  if (k < 0 || k > T) return FB4_ERR_INVALID_ARG;
  if (T == 0 || k == 0) return FB4_OK;
  if (!score || !salient_idx) return FB4_ERR_INVALID_ARG;
  cudaError_t e;
  int launches = 1;
  if (!ctx->force_generic && ctx->d_topk_scratch && fb4_topk_multi_eligible(T))
    e = fb4_launch_select_salient_topk_multi(ctx, score, T, k, salient_idx, static_cast<cudaStream_t>(stream),
                                             &launches);
  else
    e = fb4_launch_select_salient_topk(score, T, k, salient_idx, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  ctx->launches += launches;
  return FB4_OK;
}

int fb4_quantize_decomposed(fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, const float* score,
                            int32_t tile, const int32_t* cluster_id, const uint32_t* cluster_mask,
                            int32_t n_clusters, uint8_t* codes, uint16_t* meta, int32_t* salient_idx,
                            uint8_t* res_codes, uint16_t* res_meta, void* stream) {
  int rc = check_quantize_args(ctx, x, T, C, ld, codes, meta);
  if (rc != FB4_OK) return rc;
  if (tile <= 0) return FB4_ERR_INVALID_ARG;
  if (T == 0) return FB4_OK;
  if (!score || !salient_idx || !res_codes || !res_meta) return FB4_ERR_INVALID_ARG;
  if (cluster_id && (!cluster_mask || n_clusters <= 0)) return FB4_ERR_INVALID_ARG;
  if (!aligned16(res_codes) || !aligned16(res_meta)) return FB4_ERR_ALIGN;
  rc = fb4_select_salient(ctx, score, T, tile, salient_idx, stream);
  if (rc != FB4_OK) return rc;
  Fb4RowExtras ex{};
  ex.cluster_id = cluster_id;
  ex.cluster_mask = cluster_id ? cluster_mask : nullptr;
  ex.n_clusters = cluster_id ? n_clusters : 0;
  ex.salient_idx = salient_idx;
  ex.n_salient = (T + tile - 1) / tile;
  ex.tile = tile;
  ex.res_codes = res_codes;
  ex.res_meta = res_meta;
  return run_quantize(ctx, x, T, C, ld, ex, codes, meta, static_cast<cudaStream_t>(stream));
}

int fb4_quantize_decomposed_idx(fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld,
                                const int32_t* salient_idx, int64_t n_salient, const int32_t* cluster_id,
                                const uint32_t* cluster_mask, int32_t n_clusters, uint8_t* codes, uint16_t* meta,
                                uint8_t* res_codes, uint16_t* res_meta, void* stream) {
  const int rc = check_quantize_args(ctx, x, T, C, ld, codes, meta);
  if (rc != FB4_OK) return rc;
  if (n_salient < 0 || n_salient > T) return FB4_ERR_INVALID_ARG;
  if (T == 0) return FB4_OK;
  if (n_salient > 0 && (!salient_idx || !res_codes || !res_meta)) return FB4_ERR_INVALID_ARG;
  if (cluster_id && (!cluster_mask || n_clusters <= 0)) return FB4_ERR_INVALID_ARG;
  if (n_salient > 0 && (!aligned16(res_codes) || !aligned16(res_meta))) return FB4_ERR_ALIGN;
  Fb4RowExtras ex{};
  ex.cluster_id = cluster_id;
  ex.cluster_mask = cluster_id ? cluster_mask : nullptr;
  ex.n_clusters = cluster_id ? n_clusters : 0;
  ex.salient_idx = salient_idx;
  ex.n_salient = n_salient;
  ex.tile = 0;
  ex.res_codes = res_codes;
  ex.res_meta = res_meta;
  return run_quantize(ctx, x, T, C, ld, ex, codes, meta, static_cast<cudaStream_t>(stream));
}

int fb4_dequantize(fb4_ctx* ctx, const uint8_t* codes, const uint16_t* meta, int64_t T, int64_t C,
                   const int32_t* salient_idx, int64_t n_salient, const uint8_t* res_codes,
                   const uint16_t* res_meta, void* out, int out_dtype, void* stream) {
  if (!ctx) return FB4_ERR_INVALID_ARG;
  if (T < 0 || C <= 0 || C % ctx->cfg.block_size != 0 || T > 0x7fffffffLL) return FB4_ERR_SHAPE;
  if (out_dtype < 0 || out_dtype > 2) return FB4_ERR_INVALID_ARG;
  if (n_salient < 0) return FB4_ERR_INVALID_ARG;
  if (T == 0) return FB4_OK;
  if (!codes || !meta || !out) return FB4_ERR_INVALID_ARG;
  if (n_salient > 0 && (!salient_idx || !res_codes || !res_meta)) return FB4_ERR_INVALID_ARG;
  if (!aligned16(codes) || !aligned16(meta) || !aligned16(out)) return FB4_ERR_ALIGN;
  if (n_salient > 0 && (!aligned16(res_codes) || !aligned16(res_meta))) return FB4_ERR_ALIGN;
  int launches = 0;
  cudaError_t e = fb4_launch_dequantize(ctx, codes, meta, T, C, salient_idx, n_salient, res_codes, res_meta, out,
                                        out_dtype, static_cast<cudaStream_t>(stream), &launches);
  ctx->launches += launches;
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  return FB4_OK;
}

int fb4_build_subformatbook(fb4_ctx* ctx, const uint16_t* meta, int64_t T, int64_t C, const int32_t* anchor_token,
                            const int32_t* anchor_cluster, int64_t n_anchor, int32_t n_clusters, uint32_t* counts,
                            uint32_t* cluster_mask, void* stream) {
  if (!ctx) return FB4_ERR_INVALID_ARG;
  if (T < 0 || C <= 0 || C % ctx->cfg.block_size != 0 || T > 0x7fffffffLL) return FB4_ERR_SHAPE;
  if (n_anchor < 0 || n_clusters < 0) return FB4_ERR_INVALID_ARG;
  if (n_clusters == 0) return FB4_OK;
  if (!counts || !cluster_mask) return FB4_ERR_INVALID_ARG;
  if (n_anchor > 0 && (!meta || !anchor_token || !anchor_cluster)) return FB4_ERR_INVALID_ARG;
  const int64_t nblk = C / ctx->cfg.block_size;
  if (n_anchor > 0 && n_anchor > 0xffffffffLL / nblk) return FB4_ERR_SHAPE;   // counts are 32-bit
  Fb4Stage1 s1;
  std::memcpy(s1.m, ctx->host_tables.stage1, sizeof s1.m);
  int launches = 0;
  cudaError_t e = fb4_launch_subformatbook(meta, T, nblk, anchor_token, anchor_cluster, n_anchor, n_clusters, s1,
                                           counts, cluster_mask, ctx->sm_count, static_cast<cudaStream_t>(stream),
                                           &launches);
  ctx->launches += launches;
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  return FB4_OK;
}

int fb4_quantize_weights(fb4_ctx* ctx, const void* w, int64_t N, int64_t K, int64_t ld, uint8_t* codes, uint16_t* meta,
                         void* stream) {
  const int rc = check_quantize_args(ctx, w, N, K, ld, codes, meta);
  if (rc != FB4_OK) return rc;
  if (N == 0) return FB4_OK;
  cudaError_t e = fb4_launch_quantize_weights(ctx, w, N, K, ld, codes, meta, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  ctx->launches += 1;
  return FB4_OK;
}

int fb4_quantize_mxfp8(fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, const int32_t* cluster_id,
                       const uint32_t* cluster_mask, int32_t n_clusters, uint8_t* e4m3, uint8_t* scales,
                       int scale_layout, void* stream) {
  if (!ctx) return FB4_ERR_INVALID_ARG;
  if (scale_layout != 0 && scale_layout != 1) return FB4_ERR_INVALID_ARG;
  if (T < 0 || C <= 0 || C % 64 != 0 || ld < C || T > 0x7fffffffLL) return FB4_ERR_SHAPE;
  if (T == 0) return FB4_OK;
  if (!x || !e4m3 || !scales) return FB4_ERR_INVALID_ARG;
  if (cluster_id && (!cluster_mask || n_clusters <= 0)) return FB4_ERR_INVALID_ARG;
  if (!aligned16(x) || (ld & 7) || (reinterpret_cast<uintptr_t>(e4m3) & 31u)) return FB4_ERR_ALIGN;
  if (!fb4_fast_mx_eligible(ctx, x, T, C, ld)) return FB4_ERR_INVALID_ARG;   // default configuration only
  Fb4RowExtras ex{};
  ex.cluster_id = cluster_id;
  ex.cluster_mask = cluster_id ? cluster_mask : nullptr;
  ex.n_clusters = cluster_id ? n_clusters : 0;
  int launches = 0;
  cudaError_t e = fb4_launch_quantize_fast_mx(ctx, x, T, C, ld, ex, e4m3, scales, nullptr, nullptr, scale_layout,
                                              static_cast<cudaStream_t>(stream), &launches);
  ctx->launches += launches;
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  ctx->last_variant = "fast";
  return FB4_OK;
}

int fb4_quantize_mxfp8_decomposed(fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, const float* score,
                                  int32_t tile, int32_t* salient_idx, int64_t n_salient, const int32_t* cluster_id,
                                  const uint32_t* cluster_mask, int32_t n_clusters, uint8_t* e4m3, uint8_t* scales,
                                  uint8_t* res_e4m3, uint8_t* res_scales, int scale_layout, void* stream) {
  if (!ctx) return FB4_ERR_INVALID_ARG;
  if (scale_layout != 0 && scale_layout != 1) return FB4_ERR_INVALID_ARG;
  if (T < 0 || C <= 0 || C % 64 != 0 || ld < C || T > 0x7fffffffLL) return FB4_ERR_SHAPE;
  if (score ? tile <= 0 : (n_salient < 0 || n_salient > T)) return FB4_ERR_INVALID_ARG;
  if (T == 0) return FB4_OK;
  if (score) n_salient = (T + tile - 1) / tile;
  if (!x || !e4m3 || !scales) return FB4_ERR_INVALID_ARG;
  if (n_salient > 0 && (!salient_idx || !res_e4m3 || !res_scales)) return FB4_ERR_INVALID_ARG;
  if (cluster_id && (!cluster_mask || n_clusters <= 0)) return FB4_ERR_INVALID_ARG;
  if (!aligned16(x) || (ld & 7) || (reinterpret_cast<uintptr_t>(e4m3) & 31u)) return FB4_ERR_ALIGN;
  if (n_salient > 0 && (reinterpret_cast<uintptr_t>(res_e4m3) & 31u)) return FB4_ERR_ALIGN;
  if (!fb4_fast_mx_eligible(ctx, x, T, C, ld)) return FB4_ERR_INVALID_ARG;   // default configuration only
  if (score) {
    const int rc = fb4_select_salient(ctx, score, T, tile, salient_idx, stream);
    if (rc != FB4_OK) return rc;
  }
  Fb4RowExtras ex{};
  ex.cluster_id = cluster_id;
  ex.cluster_mask = cluster_id ? cluster_mask : nullptr;
  ex.n_clusters = cluster_id ? n_clusters : 0;
  ex.salient_idx = salient_idx;
  ex.n_salient = n_salient;
  ex.tile = score ? tile : 0;
  int launches = 0;
  cudaError_t e = fb4_launch_quantize_fast_mx(ctx, x, T, C, ld, ex, e4m3, scales, res_e4m3, res_scales, scale_layout,
                                              static_cast<cudaStream_t>(stream), &launches);
  ctx->launches += launches;
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  ctx->last_variant = "fast";
  return FB4_OK;
}

int64_t fb4_mxfp8_scale_bytes(int64_t T, int64_t C, int layout) {
  if (T < 0 || C <= 0 || C % 32 != 0 || (layout != 0 && layout != 1)) return -1;
  const int64_t n_col = C / 32;
  return layout == 0 ? T * n_col : ((T + 127) / 128) * ((n_col + 3) / 4) * 512;
}

int fb4_to_mxfp8(fb4_ctx* ctx, const uint8_t* codes, const uint16_t* meta, int64_t T, int64_t C, uint8_t* e4m3,
                 uint8_t* scales, int scale_layout, void* stream) {
  if (!ctx || ctx->cfg.block_size != 32) return FB4_ERR_INVALID_ARG;   // an MX block is 32 elements
  if (scale_layout != 0 && scale_layout != 1) return FB4_ERR_INVALID_ARG;
  if (T < 0 || C <= 0 || C % 32 != 0 || T > 0x7fffffffLL) return FB4_ERR_SHAPE;
  if (T == 0) return FB4_OK;
  if (!codes || !meta || !e4m3 || !scales) return FB4_ERR_INVALID_ARG;
  if (!aligned16(codes) || !aligned16(meta) || !aligned16(e4m3)) return FB4_ERR_ALIGN;
  cudaError_t e = fb4_launch_to_mxfp8(ctx, codes, meta, T, C, e4m3, scales, scale_layout,
                                      static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  ctx->launches += 1;
  return FB4_OK;
}

int fb4_quantize_host(fb4_ctx* ctx, const void* x_host, int64_t T, int64_t C, void* d_x, uint8_t* d_codes,
                      uint16_t* d_meta, uint8_t* codes_host, uint16_t* meta_host) {
  const int rc = check_quantize_args(ctx, d_x, T, C, C, d_codes, d_meta);
  if (rc != FB4_OK) return rc;
  if (T == 0) return FB4_OK;
  if (!x_host || !codes_host || !meta_host) return FB4_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return fb4_set_cuda_error(cudaGetLastError());
  for (int i = 0; i < 3; ++i) {
    if (!ctx->pipe_stream[i]) {
      cudaError_t e = cudaStreamCreateWithFlags(&ctx->pipe_stream[i], cudaStreamNonBlocking);
      if (e != cudaSuccess) return fb4_set_cuda_error(e);
    }
  }
  const int64_t nblk = C / ctx->cfg.block_size;
  // row chunks of about 16 MB of input, a multiple of 8 rows so every chunk stays 16-byte aligned
  int64_t rows = (16ll << 20) / (C * 2);
  rows = rows < 8 ? 8 : (rows & ~7ll);
  int k = 0;
  for (int64_t r0 = 0; r0 < T; r0 += rows, ++k) {
    const int64_t nr = r0 + rows < T ? rows : T - r0;
    cudaStream_t s = ctx->pipe_stream[k % 3];
    const char* xh = static_cast<const char*>(x_host) + r0 * C * 2;
    char* xd = static_cast<char*>(d_x) + r0 * C * 2;
    cudaError_t e = cudaMemcpyAsync(xd, xh, (size_t)(nr * C * 2), cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return fb4_set_cuda_error(e);
    Fb4RowExtras ex{};
    const int q = run_quantize(ctx, xd, nr, C, C, ex, d_codes + r0 * (C / 2), d_meta + r0 * nblk, s);
    if (q != FB4_OK) return q;
    e = cudaMemcpyAsync(codes_host + r0 * (C / 2), d_codes + r0 * (C / 2), (size_t)(nr * (C / 2)),
                        cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(meta_host + r0 * nblk, d_meta + r0 * nblk, (size_t)(nr * nblk * 2),
                          cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return fb4_set_cuda_error(e);
  }
  for (int i = 0; i < 3; ++i) {
    cudaError_t e = cudaStreamSynchronize(ctx->pipe_stream[i]);
    if (e != cudaSuccess) return fb4_set_cuda_error(e);
  }
  return FB4_OK;
}

int fb4_set_kernel_variant(fb4_ctx* ctx, int variant) {
  if (!ctx || variant < 0 || variant > 1) return FB4_ERR_INVALID_ARG;
  ctx->force_generic = variant;
  return FB4_OK;
}

int fb4_device_status(fb4_ctx* ctx, uint32_t* status) {
  if (!ctx || !status) return FB4_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  cudaError_t e = cudaMemcpy(status, ctx->d_status, sizeof(uint32_t), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  return FB4_OK;
}

int64_t fb4_launch_count(const fb4_ctx* ctx) { return ctx ? ctx->launches : 0; }

const char* fb4_last_variant(const fb4_ctx* ctx) { return ctx ? ctx->last_variant : "none"; }

int fb4_last_cuda_error(void) { return g_last_cuda_error.load(); }

const char* fb4_strerror(int code) {
  switch (code) {
    case FB4_OK: return "ok";
    case FB4_ERR_INVALID_ARG: return "invalid argument";
    case FB4_ERR_SHAPE: return "invalid shape";
    case FB4_ERR_ALIGN: return "misaligned pointer or leading dimension";
    case FB4_ERR_FORMATBOOK: return "invalid formatbook";
    case FB4_ERR_CUDA: return "CUDA runtime error";
    case FB4_ERR_NO_DEVICE: return "no usable sm_100 CUDA device";
    case FB4_ERR_STATIC_LIMIT: return "more clusters than the built-in scratch holds (FB4_STATIC_MAX_CLUSTERS)";
    default: return "unknown error";
  }
}

}  // extern "C"
