// Offline weight quantization (Sec. 3.3: exhaustive dialect search ahead of inference; App. C: the
// squared error is the criterion): for every block the squared error of every
// one of the 32 dialects over all elements, in double precision and in element order (so that the
// minimum is decided exactly as the definition's sequential sum decides it), the smallest wins, ties
// to the lowest id.  One thread per block; not a bandwidth path (about 3 K fp64 operations per block).
#include "fb4_internal.h"

namespace {

struct WeightTables {
  double mag[32][8];        // formatbook as doubles
  uint8_t qvalue[32][32];   // [dialect][bin] -> index of the nearest magnitude (exact, Sec. 3.2)
};

template <int B>
__global__ void __launch_bounds__(128)
fb4_quantize_weights_kernel(const uint16_t* __restrict__ w, int64_t N, int64_t K, int64_t ld,
                            const Fb4DeviceTables* __restrict__ tables, int exp_min, int exp_max,
                            uint8_t* __restrict__ codes, uint16_t* __restrict__ meta) {
  __shared__ WeightTables tb;
  for (int i = threadIdx.x; i < 256; i += blockDim.x) tb.mag[i >> 3][i & 7] = (double)tables->formatbook[i >> 3][i & 7];
  for (int i = threadIdx.x; i < 1024; i += blockDim.x) tb.qvalue[i >> 5][i & 31] = tables->qvalue[i >> 5][i & 31];
  __syncthreads();
  const int64_t nblk = K / B, total = N * nblk;
  for (int64_t id = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; id < total; id += (int64_t)gridDim.x * blockDim.x) {
    const int64_t n = id / nblk, blk = id - n * nblk;
    const uint4* src = reinterpret_cast<const uint4*>(w + n * ld + blk * B);
    float ax[B];
    uint32_t sgn = 0;
#pragma unroll
    for (int q = 0; q < B / 8; ++q) {
      const uint4 v4 = src[q];
      const uint32_t ww[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        ax[q * 8 + 2 * j] = __uint_as_float((ww[j] << 16) & 0x7fffffffu);
        ax[q * 8 + 2 * j + 1] = __uint_as_float(ww[j] & 0x7fff0000u);
        sgn |= ((ww[j] >> 15) & 1u) << (q * 8 + 2 * j);
        sgn |= (ww[j] >> 31) << (q * 8 + 2 * j + 1);
      }
    }
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < B; ++i) amax = fmaxf(amax, ax[i]);
    int e = amax == 0.f ? exp_min : (int)((__float_as_uint(amax) >> 23) & 0xff) - 127;   // subnormals: field 0 -> clamped
    e = max(exp_min, min(exp_max, e));
    // v = |x| * 2^(3-e) exactly, as a double (the product can underflow fp32)
    const double s = __longlong_as_double((long long)(1023 + 3 - e) << 52);
    double v[B];
    uint8_t bin[B];
#pragma unroll
    for (int i = 0; i < B; ++i) {
      v[i] = (double)ax[i] * s;
      bin[i] = (uint8_t)min(31, (int)(2.0 * v[i]));   // floor: v >= 0
    }
    int best = 0;
    double best_err = 0.0;
    for (int d = 0; d < 32; ++d) {
      double err = 0.0;
#pragma unroll
      for (int i = 0; i < B; ++i) {
        const double diff = __dsub_rn(v[i], tb.mag[d][tb.qvalue[d][bin[i]]]);
        err = __dadd_rn(err, __dmul_rn(diff, diff));   // no fused multiply-add: term, then sum, as defined
      }
      if (d == 0 || err < best_err) { best = d; best_err = err; }
    }
    uint32_t packed[B / 8];
#pragma unroll
    for (int q = 0; q < B / 8; ++q) {
      uint32_t word = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int k = q * 8 + i;
        word |= ((uint32_t)tb.qvalue[best][bin[k]] | (((sgn >> k) & 1u) << 3)) << (4 * i);
      }
      packed[q] = word;
    }
    uint8_t* crow = codes + n * (K / 2);
    if (B == 32) *reinterpret_cast<uint4*>(crow + blk * 16) = make_uint4(packed[0], packed[1], packed[2 % (B / 8)], packed[3 % (B / 8)]);
    else *reinterpret_cast<uint2*>(crow + blk * 8) = make_uint2(packed[0], packed[1]);
    meta[n * nblk + blk] = (uint16_t)((e + 124) | (best << 8));
  }
}

}  // namespace

cudaError_t fb4_launch_quantize_weights(const fb4_ctx* ctx, const void* w, int64_t N, int64_t K, int64_t ld,
                                        uint8_t* codes, uint16_t* meta, cudaStream_t stream) {
  const int B = (int)ctx->cfg.block_size;
  const int64_t total = N * (K / B);
  if (total == 0) return cudaSuccess;
  const int threads = 128;
  const int64_t want = (total + threads - 1) / threads, cap = (int64_t)ctx->sm_count * 16;
  const unsigned grid = (unsigned)(want < cap ? want : cap);
  const uint16_t* wp = static_cast<const uint16_t*>(w);
  if (B == 32)
    fb4_quantize_weights_kernel<32><<<grid, threads, 0, stream>>>(wp, N, K, ld, ctx->d_tables, ctx->cfg.exp_min,
                                                                 ctx->cfg.exp_max, codes, meta);
  else
    fb4_quantize_weights_kernel<16><<<grid, threads, 0, stream>>>(wp, N, K, ld, ctx->d_tables, ctx->cfg.exp_min,
                                                                 ctx->cfg.exp_max, codes, meta);
  return cudaGetLastError();
}
