// Global top-k selection of salient tokens over many CTAs (Sec. 3.3 under the reading "the k
// highest-scoring tokens of the whole sequence", ties to the lowest index, ascending output): a
// two-digit radix select on order-preserving 32-bit keys with 65 536-bin histograms in a scratch
// buffer of the context, then an ordered compaction.  Seven small stream-ordered launches, no CTA
// waits on another:
//   clear | histogram of the high 16 key bits | pick the high digit | histogram of the low 16 bits
//   among keys with that high digit | pick the low digit (= the k-th largest key and how many keys
//   equal to it are taken) | per-CTA counts of greater / equal keys | ordered write.
// Sequences too long for the scratch take the single-CTA kernel of fb4_decode.cu.
#include "fb4_internal.h"

namespace {

constexpr int kBins = 1 << 16;
constexpr int kThreads = 1024;
constexpr int kChunk = 4096;                 // elements per CTA of the count / write kernels
constexpr int64_t kMaxChunks = 4096;         // scratch holds this many per-CTA counts (T <= 16 Mi)

// scratch layout (uint32 words): hist_hi[65536] | hist_lo[65536] | state[4] | counts[2 * kMaxChunks]
constexpr size_t kStateOff = 2 * (size_t)kBins;
constexpr size_t kCountsOff = kStateOff + 4;
constexpr size_t kScratchWords = kCountsOff + 2 * (size_t)kMaxChunks;
// state: [0] high digit, [1] how many of the k are left for that digit, [2] k-th key, [3] quota of ties

__device__ __forceinline__ uint32_t score_key(float f) {   // order-preserving; -0 counts as +0
  uint32_t u = __float_as_uint(f);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// One histogram update per distinct bin of a warp (scores share their leading bits, and tie groups
// share all of them: unaggregated, the updates of one address serialize).  All lanes take part.
__device__ __forceinline__ void warp_hist_add(uint32_t* hist, uint32_t bin, bool counts) {
  const uint32_t peers = __match_any_sync(0xffffffffu, counts ? bin : 0xffffffffu);
  if (counts && (threadIdx.x & 31) == (uint32_t)(__ffs((int)peers) - 1)) atomicAdd(&hist[bin], (uint32_t)__popc(peers));
}

__global__ void __launch_bounds__(256)
topk_hist_hi_kernel(const float* __restrict__ score, int64_t T, uint32_t* __restrict__ hist) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  // warp-uniform trip count: the first lane's index decides
  for (int64_t t0 = (int64_t)blockIdx.x * blockDim.x + (threadIdx.x & ~31); t0 < T; t0 += stride) {
    const int64_t t = t0 + (threadIdx.x & 31);
    const bool in = t < T;
    warp_hist_add(hist, in ? score_key(__ldg(score + t)) >> 16 : 0u, in);
  }
}

__global__ void __launch_bounds__(256)
topk_hist_lo_kernel(const float* __restrict__ score, int64_t T, const uint32_t* __restrict__ state,
                    uint32_t* __restrict__ hist) {
  const uint32_t hi = state[0];
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t t0 = (int64_t)blockIdx.x * blockDim.x + (threadIdx.x & ~31); t0 < T; t0 += stride) {
    const int64_t t = t0 + (threadIdx.x & 31);
    const uint32_t key = t < T ? score_key(__ldg(score + t)) : 0u;
    warp_hist_add(hist, key & 0xffffu, t < T && (key >> 16) == hi);
  }
}

// One CTA: the digit d (from the top) at which the running count of keys reaches `want`:
// count(bins > d) < want <= count(bins >= d).  Thread i owns bins [64 i, 64 i + 64).
// first pass (LOW = false): want = k, writes state[0] = d, state[1] = want - count(bins > d);
// second pass (LOW = true): want = state[1], writes state[2] = key, state[3] = quota.
template <bool LOW>
__global__ void __launch_bounds__(kThreads)
topk_pick_kernel(const uint32_t* __restrict__ hist, uint32_t* __restrict__ state, uint32_t k) {
  __shared__ uint32_t warp_tot[kThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t want = LOW ? state[1] : k;
  uint32_t mine = 0;
  {
    // 64 bins = 16 independent 128-bit loads
    const uint4* h4 = reinterpret_cast<const uint4*>(hist + tid * (kBins / kThreads));
#pragma unroll
    for (int b = 0; b < kBins / kThreads / 4; ++b) {
      const uint4 v = h4[b];
      mine += v.x + v.y + v.z + v.w;
    }
  }
  // suffix sums over threads: how many keys lie in the bins of the threads above this one
  uint32_t incl = mine;   // inclusive suffix sum inside the warp (towards higher lanes)
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t v = __shfl_down_sync(0xffffffffu, incl, d);
    if (lane + d < 32) incl += v;
  }
  if (lane == 0) warp_tot[warp] = incl;
  __syncthreads();
  uint32_t higher_warps = 0;
  for (int w = warp + 1; w < kThreads / 32; ++w) higher_warps += warp_tot[w];
  const uint32_t gt = incl - mine + higher_warps;   // keys in the bins owned by higher threads
  // exactly one thread holds the digit: count above its bins < want <= count including its bins
  if (gt < want && want <= gt + mine) {
    uint32_t run = gt;
    int b = kBins / kThreads - 1;
    for (; b > 0; --b) {
      const uint32_t h = hist[tid * (kBins / kThreads) + b];
      if (run + h >= want) break;
      run += h;
    }
    const uint32_t digit = (uint32_t)(tid * (kBins / kThreads) + b);
    if (LOW) {
      state[2] = (state[0] << 16) | digit;
      state[3] = want - run;            // keys equal to the k-th that are taken (lowest indices first)
    } else {
      state[0] = digit;
      state[1] = want - run;
    }
  }
}

// per chunk of kChunk elements: how many keys are greater than / equal to the k-th
__global__ void __launch_bounds__(kThreads)
topk_count_kernel(const float* __restrict__ score, int64_t T, const uint32_t* __restrict__ state,
                  uint32_t* __restrict__ counts) {
  __shared__ uint32_t sg, se;
  if (threadIdx.x == 0) { sg = 0; se = 0; }
  __syncthreads();
  const uint32_t kth = state[2];
  uint32_t g = 0, e = 0;
  const int64_t base = (int64_t)blockIdx.x * kChunk;
#pragma unroll
  for (int u = 0; u < kChunk / kThreads; ++u) {
    const int64_t t = base + u * kThreads + threadIdx.x;
    if (t < T) {
      const uint32_t key = score_key(__ldg(score + t));
      g += key > kth;
      e += key == kth;
    }
  }
  g = __reduce_add_sync(0xffffffffu, g);
  e = __reduce_add_sync(0xffffffffu, e);
  if ((threadIdx.x & 31) == 0) { atomicAdd(&sg, g); atomicAdd(&se, e); }
  __syncthreads();
  if (threadIdx.x == 0) { counts[2 * blockIdx.x] = sg; counts[2 * blockIdx.x + 1] = se; }
}

// ordered write: the chunk's base position from the counts of the chunks before it, then a block
// scan per sub-step of kThreads elements
__global__ void __launch_bounds__(kThreads)
topk_write_kernel(const float* __restrict__ score, int64_t T, const uint32_t* __restrict__ state,
                  const uint32_t* __restrict__ counts, int32_t* __restrict__ salient_idx) {
  __shared__ uint32_t s_g, s_e;
  __shared__ uint32_t warp_sums[kThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t kth = state[2], quota = state[3];
  // greater / equal keys in the chunks before this one
  uint32_t g0 = 0, e0 = 0;
  for (int c = tid; c < (int)blockIdx.x; c += kThreads) { g0 += counts[2 * c]; e0 += counts[2 * c + 1]; }
  g0 = __reduce_add_sync(0xffffffffu, g0);
  e0 = __reduce_add_sync(0xffffffffu, e0);
  if (tid == 0) { s_g = 0; s_e = 0; }
  __syncthreads();
  if (lane == 0) { atomicAdd(&s_g, g0); atomicAdd(&s_e, e0); }
  __syncthreads();
  uint32_t g_before = s_g, e_before = s_e;   // uniform over the CTA
  const int64_t base = (int64_t)blockIdx.x * kChunk;
  for (int u = 0; u < kChunk / kThreads; ++u) {
    const int64_t t = base + u * kThreads + tid;
    uint32_t g = 0, e = 0;
    if (t < T) {
      const uint32_t key = score_key(__ldg(score + t));
      g = key > kth;
      e = key == kth;
    }
    const uint32_t bg = __ballot_sync(0xffffffffu, g), be = __ballot_sync(0xffffffffu, e);
    const uint32_t lower = (1u << lane) - 1u;
    uint32_t gb = __popc(bg & lower), eb = __popc(be & lower);
    __syncthreads();   // warp_sums of the previous sub-step have been read
    if (lane == 0) warp_sums[warp] = (__popc(bg) << 16) | __popc(be);
    __syncthreads();
    uint32_t before = 0, total = 0;
    for (int w = 0; w < kThreads / 32; ++w) {
      const uint32_t v = warp_sums[w];
      if (w < warp) before += v;
      total += v;
    }
    gb += g_before + (before >> 16);
    eb += e_before + (before & 0xffffu);
    // position = greater keys before + taken ties before (at most `quota` ties are taken, in index order)
    if (g) salient_idx[gb + min(eb, quota)] = (int32_t)t;
    else if (e && eb < quota) salient_idx[gb + eb] = (int32_t)t;
    g_before += total >> 16;
    e_before += total & 0xffffu;
  }
}

}  // namespace

size_t fb4_topk_scratch_bytes() { return kScratchWords * sizeof(uint32_t); }

bool fb4_topk_multi_eligible(int64_t T) { return T >= 8192 && (T + kChunk - 1) / kChunk <= kMaxChunks; }

cudaError_t fb4_launch_select_salient_topk_multi(const fb4_ctx* ctx, const float* score, int64_t T, int64_t k,
                                                 int32_t* salient_idx, cudaStream_t stream, int* launches) {
  uint32_t* scratch = static_cast<uint32_t*>(ctx->d_topk_scratch);
  uint32_t* hist_hi = scratch;
  uint32_t* hist_lo = scratch + kBins;
  uint32_t* state = scratch + kStateOff;
  uint32_t* counts = scratch + kCountsOff;
  *launches = 0;
  cudaError_t e = cudaMemsetAsync(scratch, 0, (kStateOff + 4) * sizeof(uint32_t), stream);
  if (e != cudaSuccess) return e;
  const int64_t want = (T + 255) / 256, cap = (int64_t)ctx->sm_count * 8;
  const unsigned grid = (unsigned)(want < cap ? want : cap);
  const unsigned chunks = (unsigned)((T + kChunk - 1) / kChunk);
  topk_hist_hi_kernel<<<grid, 256, 0, stream>>>(score, T, hist_hi);
  topk_pick_kernel<false><<<1, kThreads, 0, stream>>>(hist_hi, state, (uint32_t)k);
  topk_hist_lo_kernel<<<grid, 256, 0, stream>>>(score, T, state, hist_lo);
  topk_pick_kernel<true><<<1, kThreads, 0, stream>>>(hist_lo, state, (uint32_t)k);
  topk_count_kernel<<<chunks, kThreads, 0, stream>>>(score, T, state, counts);
  topk_write_kernel<<<chunks, kThreads, 0, stream>>>(score, T, state, counts, salient_idx);
  e = cudaGetLastError();
  if (e == cudaSuccess) *launches = 6;
  return e;
}
