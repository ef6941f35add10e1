// MXFP8 view of an FB4 tensor (App. D.2: the integer magnitudes 0..15 are exact in FP8 e4m3 and the
// block scale is a power of two, so FB4 feeds an MXFP8 GEMM without rounding): 4-bit codes ->
// e4m3 bytes, scale bytes -> E8M0 scale factors in row-major or 128x4-tiled order.
//
// Thread <-> block of 32 elements: one 128-bit load of the codes, one 16-bit load of the metadata,
// one 256-bit store of the 32 e4m3 bytes (a warp writes 1 KB contiguous), one byte store of the scale.
// The dialect's 8 magnitudes sit in two registers as e4m3 bytes; a byte permute with four 3-bit
// indices as selector looks up four elements at once, sign bits come from sign-replicating permutes.
#include "fb4_device.cuh"
#include "fb4_internal.h"

namespace {

using fb4dev::e4m3_of_small_int;

constexpr int kThreads = 256;
constexpr int kUnroll = 4;

__global__ void __launch_bounds__(kThreads)
fb4_to_mxfp8_kernel(const uint4* __restrict__ codes, const uint16_t* __restrict__ meta, int64_t T, int64_t n_col,
                    const Fb4DeviceTables* __restrict__ tables, uint8_t* __restrict__ e4m3,
                    uint8_t* __restrict__ scales, int tiled, int out_aligned32) {
  __shared__ uint2 fb8[32];   // per dialect: its 8 magnitudes as e4m3 bytes
  reinterpret_cast<uint8_t*>(fb8)[threadIdx.x] =
      (uint8_t)e4m3_of_small_int(tables->formatbook[threadIdx.x >> 3][threadIdx.x & 7]);
  __syncthreads();
  const int64_t total = T * n_col;
  const int64_t col_tiles = (n_col + 3) >> 2;
  const bool small = total < 0xffffffffLL;   // block indices fit 32 bits: row/column by 32-bit division
  constexpr int64_t kStep = (int64_t)kThreads * kUnroll;
  const int64_t stride = (int64_t)gridDim.x * kStep;
  uint4 cw[kUnroll];
  uint32_t m[kUnroll];
  auto load = [&](int64_t base) {
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int64_t b = base + u * kThreads + threadIdx.x;
      if (b < total) {
        cw[u] = __ldg(codes + b);
        m[u] = (uint32_t)__ldg(meta + b);
      }
    }
  };
  int64_t base = (int64_t)blockIdx.x * kStep;
  if (base < total) load(base);
  for (; base < total; base += stride) {
    uint4 c[kUnroll];
    uint32_t mm[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      c[u] = cw[u];
      mm[u] = m[u];
    }
    if (base + stride < total) load(base + stride);   // the next step's loads fly while this one is converted
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int64_t b = base + u * kThreads + threadIdx.x;
      if (b >= total) continue;
      const uint2 fb = fb8[(mm[u] >> 8) & 31u];
      uint32_t o[8];
      fb4dev::codes_to_e4m3(c[u].x, fb, o[0], o[1]);
      fb4dev::codes_to_e4m3(c[u].y, fb, o[2], o[3]);
      fb4dev::codes_to_e4m3(c[u].z, fb, o[4], o[5]);
      fb4dev::codes_to_e4m3(c[u].w, fb, o[6], o[7]);
      uint8_t* dst = e4m3 + b * 32;
      if (out_aligned32) {
        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(o[0]), "r"(o[1]),
                     "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
      } else {
        reinterpret_cast<uint4*>(dst)[0] = make_uint4(o[0], o[1], o[2], o[3]);
        reinterpret_cast<uint4*>(dst)[1] = make_uint4(o[4], o[5], o[6], o[7]);
      }
      int64_t off = b;   // row-major: the block index itself
      if (tiled) {
        int64_t row, col;
        if (small) {
          const uint32_t r32 = (uint32_t)b / (uint32_t)n_col;
          row = r32;
          col = (uint32_t)b - r32 * (uint32_t)n_col;
        } else {
          row = b / n_col;
          col = b - row * n_col;
        }
        off = fb4dev::mx_scale_offset(row, col, n_col, col_tiles, 1);
      }
      scales[off] = (uint8_t)mm[u];   // E8M0 of 2^(e-3)
    }
  }
  if (tiled) {
    // padding of the tiled layout holds scale 1: rows [T, Tp) x all padded columns, then rows [0, T)
    // x columns [n_col, n_col_p)
    const int64_t Tp = (T + 127) & ~127ll, n_col_p = col_tiles * 4;
    const int64_t pad_a = (Tp - T) * n_col_p, pad_b = T * (n_col_p - n_col);
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < pad_a + pad_b;
         i += (int64_t)gridDim.x * kThreads) {
      int64_t row, col;
      if (i < pad_a) {
        row = T + i / n_col_p;
        col = i % n_col_p;
      } else {
        const int64_t j = i - pad_a, w = n_col_p - n_col;
        row = j / w;
        col = n_col + j % w;
      }
      scales[fb4dev::mx_scale_offset(row, col, n_col, col_tiles, 1)] = 0x7f;
    }
  }
}

// Tiled scale order, scales 16-byte aligned: a CTA takes 128 rows x 32 block columns at a time (the
// rows of one scale tile, eight column tiles wide), each warp a row segment of 32 blocks per step,
// and gathers the 4 KB of scale bytes of those eight tiles in shared memory in their final order;
// the tiles are contiguous in the output, so the CTA then writes them as whole 16-byte pieces.  (With
// one byte store per block, as in the kernel above, every 32-byte sector of the scale array is
// written by eight separate requests.)  Padding bytes (scale 1) come from the same pass.
constexpr int kTileStride = 528;   // 512 bytes of a scale tile + 16: the eight tiles start in different banks

__global__ void __launch_bounds__(kThreads)
fb4_to_mxfp8_tiled_kernel(const uint4* __restrict__ codes, const uint16_t* __restrict__ meta, int64_t T, int64_t n_col,
                          const Fb4DeviceTables* __restrict__ tables, uint8_t* __restrict__ e4m3,
                          uint8_t* __restrict__ scales, int out_aligned32) {
  __shared__ uint2 fb8[32];
  __shared__ __align__(16) uint8_t sc[8 * kTileStride];
  reinterpret_cast<uint8_t*>(fb8)[threadIdx.x] =
      (uint8_t)e4m3_of_small_int(tables->formatbook[threadIdx.x >> 3][threadIdx.x & 7]);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t row_tiles = (T + 127) >> 7, col_chunks = (n_col + 31) >> 5, col_tiles = (n_col + 3) >> 2;
  const int64_t items = row_tiles * col_chunks;
  for (int64_t it = blockIdx.x; it < items; it += gridDim.x) {
    const int64_t rt = it / col_chunks, cc = it - rt * col_chunks;
    const int64_t col = cc * 32 + lane;
    const bool col_ok = col < n_col;
    __syncthreads();   // fb8 is filled; the previous item's scale bytes have been written out
#pragma unroll 1
    for (int g = 0; g < 4; ++g) {
      uint4 c[4];
      uint32_t m[4];
      bool ok[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int64_t row = rt * 128 + warp + 8 * (g * 4 + u);
        ok[u] = col_ok && row < T;
        m[u] = 0x7fu;   // padding: scale 1
        c[u] = make_uint4(0u, 0u, 0u, 0u);
        if (ok[u]) {
          const int64_t b = row * n_col + col;
          c[u] = __ldg(codes + b);
          m[u] = (uint32_t)__ldg(meta + b);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int rr = warp + 8 * (g * 4 + u);
        sc[(lane >> 2) * kTileStride + (rr & 31) * 16 + (rr >> 5) * 4 + (lane & 3)] = (uint8_t)m[u];
        if (!ok[u]) continue;
        const uint2 fb = fb8[(m[u] >> 8) & 31u];
        uint32_t o[8];
        fb4dev::codes_to_e4m3(c[u].x, fb, o[0], o[1]);
        fb4dev::codes_to_e4m3(c[u].y, fb, o[2], o[3]);
        fb4dev::codes_to_e4m3(c[u].z, fb, o[4], o[5]);
        fb4dev::codes_to_e4m3(c[u].w, fb, o[6], o[7]);
        uint8_t* dst = e4m3 + ((rt * 128 + rr) * n_col + col) * 32;
        if (out_aligned32) {
          asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(o[0]), "r"(o[1]),
                       "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
        } else {
          reinterpret_cast<uint4*>(dst)[0] = make_uint4(o[0], o[1], o[2], o[3]);
          reinterpret_cast<uint4*>(dst)[1] = make_uint4(o[4], o[5], o[6], o[7]);
        }
      }
    }
    __syncthreads();
    // eight tiles x 512 bytes = 256 threads x 16 bytes; column tiles past the last one do not exist
    const int64_t ct = cc * 8 + warp;
    if (ct < col_tiles)
      *reinterpret_cast<uint4*>(scales + (rt * col_tiles + ct) * 512 + lane * 16) =
          *reinterpret_cast<const uint4*>(sc + warp * kTileStride + lane * 16);
  }
}

}  // namespace

cudaError_t fb4_launch_to_mxfp8(const fb4_ctx* ctx, const uint8_t* codes, const uint16_t* meta, int64_t T, int64_t C,
                                uint8_t* e4m3, uint8_t* scales, int layout, cudaStream_t stream) {
  static_assert(kThreads == 256, "one thread per formatbook entry fills the shared table");
  const int64_t n_col = C / 32, total = T * n_col;
  if (total == 0) return cudaSuccess;
  constexpr int64_t kStep = (int64_t)kThreads * kUnroll;
  const int64_t want = (total + kStep - 1) / kStep, cap = 0x7fffffff;   // one step per CTA (see fb4_decode.cu)
  const int a32 = (reinterpret_cast<uintptr_t>(e4m3) & 31u) == 0 ? 1 : 0;
  if (layout == 1 && (reinterpret_cast<uintptr_t>(scales) & 15u) == 0) {
    const int64_t items = ((T + 127) >> 7) * ((n_col + 31) >> 5);
    fb4_to_mxfp8_tiled_kernel<<<(unsigned)(items < cap ? items : cap), kThreads, 0, stream>>>(
        reinterpret_cast<const uint4*>(codes), meta, T, n_col, ctx->d_tables, e4m3, scales, a32);
    return cudaGetLastError();
  }
  fb4_to_mxfp8_kernel<<<(unsigned)(want < cap ? want : cap), kThreads, 0, stream>>>(
      reinterpret_cast<const uint4*>(codes), meta, T, n_col, ctx->d_tables, e4m3, scales, layout, a32);
  return cudaGetLastError();
}
