// Global top-k selection of salient tokens over many CTAs (Sec. 3.3 under the reading "the k
// highest-scoring tokens of the whole sequence", ties to the lowest index, ascending output): a
// two-digit radix select on order-preserving 32-bit keys with 65 536-bin histograms in a scratch
// buffer of the context, then an ordered compaction.  Five small stream-ordered launches, no CTA
// waits on another:
//   clear | histogram of the high 16 key bits, and the CTA that finishes last picks the high digit |
//   histogram of the low 16 bits among keys with that high digit, and the last CTA picks the low
//   digit (= the k-th largest key and how many keys equal to it are taken) | per-CTA counts of
//   greater / equal keys | ordered write.
// Sequences too long for the scratch take the single-CTA kernel of fb4_decode.cu.
#include "fb4_internal.h"

namespace {

constexpr int kBins = 1 << 16;
constexpr int kThreads = 1024;
constexpr int kChunk = 4096;                 // elements per CTA of the count / write kernels
constexpr int64_t kMaxChunks = 4096;         // scratch holds this many per-CTA counts (T <= 16 Mi)

// scratch layout (uint32 words): hist_hi[65536] | hist_lo[65536] | state[8] | counts[2 * kMaxChunks]
constexpr size_t kStateOff = 2 * (size_t)kBins;
constexpr size_t kStateWords = 8;
constexpr size_t kCountsOff = kStateOff + kStateWords;
constexpr size_t kScratchWords = kCountsOff + 2 * (size_t)kMaxChunks;
// state: [0] high digit, [1] how many of the k are left for that digit, [2] k-th key, [3] quota of ties,
//        [4] / [5] CTAs that have finished the high / low histogram

__device__ __forceinline__ uint32_t score_key(float f) {   // order-preserving; -0 counts as +0
  uint32_t u = __float_as_uint(f);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kHistThreads = 256;    // also the width of the digit pick by the last CTA

// inclusive suffix sum over the CTA's kHistThreads threads (towards higher thread ids)
__device__ __forceinline__ uint32_t cta_suffix_sum(uint32_t v, uint32_t* warp_tot) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t incl = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t o = __shfl_down_sync(0xffffffffu, incl, d);
    if (lane + d < 32) incl += o;
  }
  __syncthreads();            // warp_tot of an earlier call has been read
  if (lane == 0) warp_tot[warp] = incl;
  __syncthreads();
  for (int w = warp + 1; w < kHistThreads / 32; ++w) incl += warp_tot[w];
  return incl;
}

// One CTA of kHistThreads threads: the digit d (from the top) at which the running count of keys
// reaches `want`: count(bins > d) < want <= count(bins >= d).  Two parallel steps: which thread's
// 256 bins hold it, then which of those bins.  The histogram was written by atomics of other CTAs:
// read it from L2.
// first digit (LOW = false): want = k, writes state[0] = d, state[1] = want - count(bins > d);
// second digit (LOW = true): want = state[1], writes state[2] = key, state[3] = quota.
template <bool LOW>
__device__ __forceinline__ void pick_digit(const uint32_t* hist, uint32_t* state, uint32_t k) {
  __shared__ uint32_t warp_tot[kHistThreads / 32];
  __shared__ uint32_t s_owner, s_above;
  const int tid = threadIdx.x;
  constexpr int kPer = kBins / kHistThreads;   // 256 bins per thread
  const uint32_t want = LOW ? __ldcg(state + 1) : k;
  uint32_t mine = 0;
  {
    const uint4* h4 = reinterpret_cast<const uint4*>(hist + tid * kPer);
#pragma unroll 16
    for (int b = 0; b < kPer / 4; ++b) {
      const uint4 v = __ldcg(h4 + b);
      mine += v.x + v.y + v.z + v.w;
    }
  }
  const uint32_t incl = cta_suffix_sum(mine, warp_tot);
  const uint32_t gt = incl - mine;                         // keys in the bins of higher threads
  if (gt < want && want <= gt + mine) { s_owner = (uint32_t)tid; s_above = gt; }   // exactly one thread
  __syncthreads();
  const uint32_t bin = s_owner * kPer + (uint32_t)tid;     // one bin of the owner's range per thread
  const uint32_t h = tid < kPer ? __ldcg(hist + bin) : 0u;
  const uint32_t incl2 = cta_suffix_sum(h, warp_tot);
  const uint32_t run = s_above + incl2 - h;                // keys above this bin
  if (run < want && want <= run + h) {
    if (LOW) {
      state[2] = (__ldcg(state + 0) << 16) | bin;
      state[3] = want - run;          // keys equal to the k-th that are taken (lowest indices first)
    } else {
      state[0] = bin;
      state[1] = want - run;
    }
  }
}

// One histogram update per distinct bin of a warp (scores share their leading bits, and tie groups
// share all of them: unaggregated, the updates of one address serialize).  All lanes take part.
__device__ __forceinline__ void warp_hist_add(uint32_t* hist, uint32_t bin, bool counts) {
  const uint32_t peers = __match_any_sync(0xffffffffu, counts ? bin : 0xffffffffu);
  if (counts && (threadIdx.x & 31) == (uint32_t)(__ffs((int)peers) - 1)) atomicAdd(&hist[bin], (uint32_t)__popc(peers));
}

// Histogram of the high (LOW = false) or, among keys with the chosen high digit, the low 16 key bits.
// The CTA whose ticket shows that all others have finished picks the digit; nobody waits.
template <bool LOW>
__global__ void __launch_bounds__(kHistThreads)
topk_hist_kernel(const float* __restrict__ score, int64_t T, uint32_t* __restrict__ hist, uint32_t* __restrict__ state,
                 uint32_t k) {
  __shared__ bool s_last;
  const uint32_t hi = LOW ? state[0] : 0u;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  // warp-uniform trip count: the first lane's index decides
  for (int64_t t0 = (int64_t)blockIdx.x * blockDim.x + (threadIdx.x & ~31); t0 < T; t0 += stride) {
    const int64_t t = t0 + (threadIdx.x & 31);
    const uint32_t key = t < T ? score_key(__ldg(score + t)) : 0u;
    if (LOW) warp_hist_add(hist, key & 0xffffu, t < T && (key >> 16) == hi);
    else warp_hist_add(hist, key >> 16, t < T);
  }
  __threadfence();            // this CTA's updates before its ticket
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(state + 4 + (LOW ? 1 : 0), 1u) == gridDim.x - 1;
  __syncthreads();
  if (s_last) {
    __threadfence();
    pick_digit<LOW>(hist, state, k);
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
  cudaError_t e = cudaMemsetAsync(scratch, 0, (kStateOff + kStateWords) * sizeof(uint32_t), stream);
  if (e != cudaSuccess) return e;
  const int64_t want = (T + kHistThreads - 1) / kHistThreads, cap = (int64_t)ctx->sm_count * 8;
  const unsigned grid = (unsigned)(want < cap ? want : cap);
  const unsigned chunks = (unsigned)((T + kChunk - 1) / kChunk);
  topk_hist_kernel<false><<<grid, kHistThreads, 0, stream>>>(score, T, hist_hi, state, (uint32_t)k);
  topk_hist_kernel<true><<<grid, kHistThreads, 0, stream>>>(score, T, hist_lo, state, (uint32_t)k);
  topk_count_kernel<<<chunks, kThreads, 0, stream>>>(score, T, state, counts);
  topk_write_kernel<<<chunks, kThreads, 0, stream>>>(score, T, state, counts, salient_idx);
  e = cudaGetLastError();
  if (e == cudaSuccess) *launches = 4;
  return e;
}
