// SeDA sub-formatbook construction (Sec. 3.4): bin-count profiling of the dialects chosen on a
// cluster's anchor tokens, then the most frequent dialect of every dynamic-range bucket.
//
// Two kernels on the caller's stream behind a memset of the count scratch:
//   count    : one warp per anchor token; a 32-bin histogram of the dialect ids of the token's
//              metadata row is built in shared memory and added to counts[cluster][dialect]
//   finalize : one thread per cluster; for every entry of the stage-1 table (a dynamic-range
//              bucket) the member with the highest count, ties to the lowest id
#include "fb4_internal.h"

namespace {

constexpr int kCountWarps = 8;

__global__ void __launch_bounds__(kCountWarps * 32)
fb4_subformatbook_count_kernel(const uint16_t* __restrict__ meta, int64_t T, int64_t nblk,
                               const int32_t* __restrict__ anchor_token, const int32_t* __restrict__ anchor_cluster,
                               int64_t n_anchor, int32_t n_clusters, uint32_t* __restrict__ counts) {
  __shared__ uint32_t hist[kCountWarps][32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int64_t a = (int64_t)blockIdx.x * kCountWarps + warp; a < n_anchor; a += (int64_t)gridDim.x * kCountWarps) {
    const int64_t tok = anchor_token[a];
    const int32_t c = anchor_cluster[a];
    if (tok < 0 || tok >= T || c < 0 || c >= n_clusters) continue;   // warp-uniform: ignored anchors
    hist[warp][lane] = 0;
    __syncwarp();
    const uint16_t* row = meta + tok * nblk;
    for (int64_t b = lane; b < nblk; b += 32) atomicAdd(&hist[warp][(row[b] >> 8) & 31u], 1u);
    __syncwarp();
    const uint32_t v = hist[warp][lane];
    if (v) atomicAdd(&counts[(int64_t)c * 32 + lane], v);
    __syncwarp();
  }
}

__global__ void fb4_subformatbook_finalize_kernel(const uint32_t* __restrict__ counts, int32_t n_clusters,
                                                  Fb4Stage1 s1, uint32_t* __restrict__ cluster_mask) {
  const int32_t c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= n_clusters) return;
  const uint32_t* cnt = counts + (int64_t)c * 32;
  uint32_t mask = 0;
  for (int k = 0; k < 32; ++k) {
    int best = -1;
    uint32_t best_count = 0;
    for (uint32_t m = s1.m[k]; m; m &= m - 1) {   // ascending ids: ties keep the lowest
      const int d = __ffs((int)m) - 1;
      const uint32_t v = cnt[d];
      if (best < 0 || v > best_count) { best = d; best_count = v; }
    }
    if (best >= 0) mask |= 1u << best;
  }
  cluster_mask[c] = mask;
}

}  // namespace

cudaError_t fb4_launch_subformatbook(const uint16_t* meta, int64_t T, int64_t nblk, const int32_t* anchor_token,
                                     const int32_t* anchor_cluster, int64_t n_anchor, int32_t n_clusters,
                                     const Fb4Stage1& stage1, uint32_t* counts, uint32_t* cluster_mask, int sm_count,
                                     cudaStream_t stream, int* launches) {
  *launches = 0;
  if (n_clusters <= 0) return cudaSuccess;
  cudaError_t e = cudaMemsetAsync(counts, 0, (size_t)n_clusters * 32 * sizeof(uint32_t), stream);
  if (e != cudaSuccess) return e;
  if (n_anchor > 0) {
    const int64_t want = (n_anchor + kCountWarps - 1) / kCountWarps;
    const int64_t cap = (int64_t)sm_count * 8;
    fb4_subformatbook_count_kernel<<<(unsigned)(want < cap ? want : cap), kCountWarps * 32, 0, stream>>>(
        meta, T, nblk, anchor_token, anchor_cluster, n_anchor, n_clusters, counts);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    *launches += 1;
  }
  fb4_subformatbook_finalize_kernel<<<(unsigned)((n_clusters + 127) / 128), 128, 0, stream>>>(counts, n_clusters, stage1,
                                                                                             cluster_mask);
  e = cudaGetLastError();
  if (e == cudaSuccess) *launches += 1;
  return e;
}
