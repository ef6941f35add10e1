// fb4_build_subformatbook_static: the sub-formatbook construction of fb4_subformatbook.cu for
// callers that may not allocate device memory.  The per-cluster dialect counts, which the
// ordinary entry point keeps in a buffer the caller allocates, live here in a fixed array that is
// part of the library image: every GPU that loads the library carries these 128 KB until the
// process exits, and every call on that GPU uses the same array.
#include <mutex>

#include "fb4_internal.h"

namespace {

// counts[cluster][dialect] for up to FB4_STATIC_MAX_CLUSTERS clusters
static __device__ __align__(256) uint32_t g_static_counts[FB4_STATIC_MAX_CLUSTERS * 32];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
uint32_t* g_counts_on_device[kMaxDevices] = {};   // device address of g_static_counts, per device ordinal

// In host code the name g_static_counts is only a handle of the symbol, not an address a kernel can
// use; the address on the current device comes from the runtime, once per device.
cudaError_t static_counts_address(int device, uint32_t** out) {
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_counts_on_device[device]) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_static_counts);
    if (e != cudaSuccess) return e;
    g_counts_on_device[device] = static_cast<uint32_t*>(p);
  }
  *out = g_counts_on_device[device];
  return cudaSuccess;
}

}  // namespace

extern "C" int fb4_build_subformatbook_static(fb4_ctx* ctx, const uint16_t* meta, int64_t T, int64_t C,
                                              const int32_t* anchor_token, const int32_t* anchor_cluster,
                                              int64_t n_anchor, int32_t n_clusters, uint32_t* cluster_mask,
                                              void* stream) {
  if (!ctx) return FB4_ERR_INVALID_ARG;
  if (T < 0 || C <= 0 || C % ctx->cfg.block_size != 0 || T > 0x7fffffffLL) return FB4_ERR_SHAPE;
  if (n_anchor < 0 || n_clusters < 0) return FB4_ERR_INVALID_ARG;
  if (n_clusters > FB4_STATIC_MAX_CLUSTERS) return FB4_ERR_STATIC_LIMIT;
  if (n_clusters == 0) return FB4_OK;
  if (!cluster_mask) return FB4_ERR_INVALID_ARG;
  if (n_anchor > 0 && (!meta || !anchor_token || !anchor_cluster)) return FB4_ERR_INVALID_ARG;
  const int64_t nblk = C / ctx->cfg.block_size;
  if (n_anchor > 0 && n_anchor > 0xffffffffLL / nblk) return FB4_ERR_SHAPE;   // counts are 32-bit
  int current = -1;
  cudaError_t e = cudaGetDevice(&current);
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  if (current != ctx->device || current < 0 || current >= kMaxDevices) return FB4_ERR_INVALID_ARG;
  uint32_t* counts = nullptr;
  e = static_counts_address(current, &counts);
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  Fb4Stage1 s1;
  for (int k = 0; k < 32; ++k) s1.m[k] = ctx->host_tables.stage1[k];
  int launches = 0;
  // the launcher clears the counts of the n_clusters clusters it uses before counting
  e = fb4_launch_subformatbook(meta, T, nblk, anchor_token, anchor_cluster, n_anchor, n_clusters, s1, counts,
                               cluster_mask, ctx->sm_count, static_cast<cudaStream_t>(stream), &launches);
  ctx->launches += launches;
  if (e != cudaSuccess) return fb4_set_cuda_error(e);
  return FB4_OK;
}
