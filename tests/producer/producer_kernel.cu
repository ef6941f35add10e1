// A producer kernel outside the library that ends in the FB4 quantizer (include/fb4_block.cuh):
// y = (x + 1) * 0.75 evaluated in fp32 (two correctly rounded operations), quantized from registers;
// y never exists in memory.  One thread per 32-element block.  Built by tests/test_gpu_block_header.py.
#include <stdint.h>

#include "fb4_block.cuh"

__global__ void producer_kernel(const void* __restrict__ image, const uint16_t* __restrict__ x, int64_t n_blocks,
                                uint8_t* __restrict__ codes, uint16_t* __restrict__ meta) {
  extern __shared__ __align__(16) unsigned char smem[];
  fb4blk::Tables* tb = reinterpret_cast<fb4blk::Tables*>(smem);
  fb4blk::copy_tables(tb, image);
  __syncthreads();
  const fb4blk::Lane ln = fb4blk::lane_state(tb);
  for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < n_blocks; b += (int64_t)gridDim.x * blockDim.x) {
    float y[32];
    const uint4* src = reinterpret_cast<const uint4*>(x + b * 32);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint4 v = src[q];
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float lo = __uint_as_float(w[j] << 16), hi = __uint_as_float(w[j] & 0xffff0000u);
        y[8 * q + 2 * j] = __fmul_rn(__fadd_rn(lo, 1.0f), 0.75f);
        y[8 * q + 2 * j + 1] = __fmul_rn(__fadd_rn(hi, 1.0f), 0.75f);
      }
    }
    uint32_t cw[4];
    uint16_t m;
    fb4blk::quantize_block_f32(y, 0xffffffffu, tb, ln, cw, &m);
    *reinterpret_cast<uint4*>(codes + b * 16) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
    meta[b] = m;
  }
}

extern "C" int producer_launch(const void* image, const void* x, int64_t n_blocks, void* codes, void* meta, void* stream) {
  const int smem = (int)sizeof(fb4blk::Tables);
  cudaError_t e = cudaFuncSetAttribute(producer_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return (int)e;
  const int threads = 256;
  int64_t grid = (n_blocks + threads - 1) / threads;
  if (grid > 296) grid = 296;
  if (grid < 1) grid = 1;
  producer_kernel<<<(int)grid, threads, smem, static_cast<cudaStream_t>(stream)>>>(
      image, static_cast<const uint16_t*>(x), n_blocks, static_cast<uint8_t*>(codes), static_cast<uint16_t*>(meta));
  return (int)cudaGetLastError();
}

extern "C" unsigned long long producer_table_bytes(void) { return sizeof(fb4blk::Tables); }
