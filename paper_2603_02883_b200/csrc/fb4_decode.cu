// FB4 decode (4-bit codes + block metadata -> fp32 / bf16, optionally adding the decoded
// residual of salient tokens) and the per-tile salient-token selection.
#include "fb4_internal.h"

namespace {

__device__ __forceinline__ float pow2f(int k) {   // 2^k, k in [-149,127]
  return k >= -126 ? __int_as_float((k + 127) << 23) : __int_as_float(1 << (k + 149));
}

__device__ __forceinline__ uint32_t f32_to_bf16_rne(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u + 0x7fffu + ((u >> 16) & 1u)) >> 16;
}

// value of one 4-bit code: (-1)^sign * magnitude * 2^(e-3); fb_lo/fb_hi = the dialect's 8 magnitudes
__device__ __forceinline__ float decode(uint32_t nib, uint32_t fb_lo, uint32_t fb_hi, float scale) {
  const uint32_t m = __byte_perm(fb_lo, fb_hi, nib & 7u) & 0xffu;
  const float v = (float)m * scale;   // exact: m <= 15, scale a power of two >= 2^-127
  return __uint_as_float(__float_as_uint(v) | ((nib & 8u) << 28));
}

constexpr int kDecodeThreads = 256;

// One CTA = one segment of kDecodeThreads code words (8 elements each) of one token row.
template <int OUT_BF16>
__global__ void __launch_bounds__(kDecodeThreads)
fb4_dequantize_kernel(const uint32_t* __restrict__ codes, const uint16_t* __restrict__ meta, int64_t T, int64_t C,
                      int block_shift, const Fb4DeviceTables* __restrict__ tables,
                      const int32_t* __restrict__ salient_idx, int64_t n_salient,
                      const uint32_t* __restrict__ res_codes, const uint16_t* __restrict__ res_meta,
                      void* __restrict__ out, int segs) {
  __shared__ uint2 fb[32];
  __shared__ int64_t s_srow;
  if (threadIdx.x < 32) fb[threadIdx.x] = reinterpret_cast<const uint2*>(tables->formatbook)[threadIdx.x];
  const int64_t t = blockIdx.x / segs;
  const int seg = (int)(blockIdx.x - t * segs);
  if (threadIdx.x == 0) {
    int64_t srow = -1, lo = 0, hi = n_salient - 1;
    while (lo <= hi) {
      const int64_t mid = (lo + hi) >> 1;
      const int32_t v = salient_idx[mid];
      if (v == (int32_t)t) { srow = mid; break; }
      if (v < (int32_t)t) lo = mid + 1; else hi = mid - 1;
    }
    s_srow = srow;
  }
  __syncthreads();
  const int64_t words = C >> 3;
  const int64_t w = (int64_t)seg * kDecodeThreads + threadIdx.x;
  if (w >= words) return;
  const int64_t nblk = C >> block_shift;
  const int64_t blk = (w << 3) >> block_shift;
  const uint32_t cw = codes[t * words + w];
  const uint32_t m = meta[t * nblk + blk];
  const uint2 d = fb[(m >> 8) & 31u];
  const float sc = pow2f((int)(m & 0xffu) - 127);
  float v[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = decode((cw >> (4 * i)) & 15u, d.x, d.y, sc);
  const int64_t srow = s_srow;
  if (srow >= 0) {
    const uint32_t rw = res_codes[srow * words + w];
    const uint32_t rm = res_meta[srow * nblk + blk];
    const uint2 rd = fb[(rm >> 8) & 31u];
    const float rs = pow2f((int)(rm & 0xffu) - 127);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __fadd_rn(v[i], decode((rw >> (4 * i)) & 15u, rd.x, rd.y, rs));
  }
  if (OUT_BF16) {
    uint4 o;
    o.x = f32_to_bf16_rne(v[0]) | (f32_to_bf16_rne(v[1]) << 16);
    o.y = f32_to_bf16_rne(v[2]) | (f32_to_bf16_rne(v[3]) << 16);
    o.z = f32_to_bf16_rne(v[4]) | (f32_to_bf16_rne(v[5]) << 16);
    o.w = f32_to_bf16_rne(v[6]) | (f32_to_bf16_rne(v[7]) << 16);
    reinterpret_cast<uint4*>(out)[t * words + w] = o;
  } else {
    float4* o = reinterpret_cast<float4*>(out) + (t * words + w) * 2;
    o[0] = make_float4(v[0], v[1], v[2], v[3]);
    o[1] = make_float4(v[4], v[5], v[6], v[7]);
  }
}

// Sec. 3.3: one salient token per tile = the highest score of the tile, ties to the lowest index.
__global__ void fb4_select_salient_kernel(const float* __restrict__ score, int64_t T, int32_t tile,
                                          int32_t* __restrict__ salient_idx, int64_t n_tiles) {
  const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= n_tiles) return;
  const int64_t t0 = k * tile;
  const int64_t t1 = t0 + tile < T ? t0 + tile : T;
  int64_t arg = t0;
  float best = score[t0];
  for (int64_t t = t0 + 1; t < t1; ++t) {
    const float s = score[t];
    if (s > best) { best = s; arg = t; }
  }
  salient_idx[k] = (int32_t)arg;
}

}  // namespace

cudaError_t fb4_launch_dequantize(const fb4_ctx* ctx, const uint8_t* codes, const uint16_t* meta, int64_t T,
                                  int64_t C, const int32_t* salient_idx, int64_t n_salient,
                                  const uint8_t* res_codes, const uint16_t* res_meta, void* out, int out_dtype,
                                  cudaStream_t stream) {
  if (T == 0 || C == 0) return cudaSuccess;
  const int64_t words = C / 8;
  const int segs = (int)((words + kDecodeThreads - 1) / kDecodeThreads);
  const int64_t grid = T * segs;
  if (grid > 0x7fffffffLL) return cudaErrorInvalidValue;
  const int shift = ctx->cfg.block_size == 32 ? 5 : 4;
  const uint32_t* cw = reinterpret_cast<const uint32_t*>(codes);
  const uint32_t* rw = reinterpret_cast<const uint32_t*>(res_codes);
  if (out_dtype == 1)
    fb4_dequantize_kernel<1><<<(unsigned)grid, kDecodeThreads, 0, stream>>>(
        cw, meta, T, C, shift, ctx->d_tables, salient_idx, n_salient, rw, res_meta, out, segs);
  else
    fb4_dequantize_kernel<0><<<(unsigned)grid, kDecodeThreads, 0, stream>>>(
        cw, meta, T, C, shift, ctx->d_tables, salient_idx, n_salient, rw, res_meta, out, segs);
  return cudaGetLastError();
}

cudaError_t fb4_launch_select_salient(const float* score, int64_t T, int32_t tile, int32_t* salient_idx,
                                      cudaStream_t stream) {
  if (T == 0) return cudaSuccess;
  const int64_t n_tiles = (T + tile - 1) / tile;
  const int threads = 128;
  fb4_select_salient_kernel<<<(unsigned)((n_tiles + threads - 1) / threads), threads, 0, stream>>>(
      score, T, tile, salient_idx, n_tiles);
  return cudaGetLastError();
}
