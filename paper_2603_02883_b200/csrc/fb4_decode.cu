// FB4 decode (4-bit codes + block metadata -> fp32 / bf16, optionally adding the decoded
// residual of salient tokens) and the per-tile salient-token selection.
#include "fb4_internal.h"

namespace {

__device__ __forceinline__ uint32_t f32_to_bf16_rne(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u + 0x7fffu + ((u >> 16) & 1u)) >> 16;
}

constexpr int kDecodeThreads = 256;
constexpr int kDecodeUnroll = 2;          // blocks in flight per thread

__device__ __forceinline__ uint32_t mul_bf16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
// prmt.b32 in its default mode (selector bit 3 of a nibble replicates the sign of the chosen byte)
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

// 32 bytes per store: a lane writes whole 32-byte sectors.  p must be 32-byte aligned when wide.
__device__ __forceinline__ void store_b32x8(void* p, const uint32_t* v, bool wide) {
  if (wide) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(v[0]), "r"(v[1]), "r"(v[2]),
                 "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]) : "memory");
  } else {
    reinterpret_cast<uint4*>(p)[0] = make_uint4(v[0], v[1], v[2], v[3]);
    reinterpret_cast<uint4*>(p)[1] = make_uint4(v[4], v[5], v[6], v[7]);
  }
}

// One code word (8 elements) -> 4 registers of two bf16 values each.
// dt = the dialect's magnitudes as bf16 bit patterns, split into a table of high bytes (x,y) and
// a table of low bytes (z,w): a byte permute with the four 3-bit indices as selector looks up
// four magnitudes at once, no memory access per element.  One packed multiply applies the scale
// sc2 (the block scale as two bf16).  Exact: a magnitude 0..15 times a power of two >= 2^-127 is
// a bf16 value (subnormals included).
__device__ __forceinline__ void decode_word(uint32_t cw, const uint4& dt, uint32_t sc2, uint32_t* pr) {
  const uint32_t sel = cw & 0x77777777u;
  const uint32_t hi_a = prmt(dt.x, dt.y, sel), lo_a = prmt(dt.z, dt.w, sel);              // elements 0..3
  const uint32_t hi_b = prmt(dt.x, dt.y, sel >> 16), lo_b = prmt(dt.z, dt.w, sel >> 16);  // elements 4..7
  // byte masks of the sign bits: bit 7 of a code byte is the sign of its odd element
  const uint32_t s_odd = prmt(cw, 0u, 0xba98u), s_even = prmt(cw << 4, 0u, 0xba98u);
  const uint32_t mag[4] = {__byte_perm(lo_a, hi_a, 0x5140), __byte_perm(lo_a, hi_a, 0x7362),
                           __byte_perm(lo_b, hi_b, 0x5140), __byte_perm(lo_b, hi_b, 0x7362)};
  const uint32_t sgn[4] = {__byte_perm(s_even, s_odd, 0x4000), __byte_perm(s_even, s_odd, 0x5010),
                           __byte_perm(s_even, s_odd, 0x6020), __byte_perm(s_even, s_odd, 0x7030)};
#pragma unroll
  for (int j = 0; j < 4; ++j) pr[j] = mul_bf16x2(mag[j], sc2) | (sgn[j] & 0x80008000u);
}

// block scale 2^(sb-127) as two bf16: sb << 7, or the subnormal 2^-127 = 0x0040 for sb = 0
__device__ __forceinline__ uint32_t scale_bf16x2(uint32_t m) {
  const uint32_t sb = m & 0xffu;
  return (sb ? (sb << 7) : 0x40u) * 0x10001u;
}

template <int WPB>
__device__ __forceinline__ void load_block_codes(const uint32_t* p, uint32_t* cw) {
  if (WPB == 4) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
    cw[0] = v.x; cw[1] = v.y; cw[2] = v.z; cw[3] = v.w;
  } else {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
    cw[0] = v.x; cw[1] = v.y;
  }
}

// 4x4 transpose of code words inside a quad of lanes: in, lane p of a quad holds the 4 words of its
// own block; out, it holds word p of the quad's blocks 0..3.  Two butterfly stages (lane xor 2,
// lane xor 1), four shuffles.  After it a quad writes whole 128-byte lines per store instruction.
__device__ __forceinline__ void quad_transpose(uint32_t (&c)[4], int lane) {
  const bool b1 = lane & 2, b0 = lane & 1;
  {
    const uint32_t s0 = b1 ? c[0] : c[2], s1 = b1 ? c[1] : c[3];
    const uint32_t r0 = __shfl_xor_sync(0xffffffffu, s0, 2), r1 = __shfl_xor_sync(0xffffffffu, s1, 2);
    if (b1) { c[0] = r0; c[1] = r1; } else { c[2] = r0; c[3] = r1; }
  }
  {
    const uint32_t s0 = b0 ? c[0] : c[1], s1 = b0 ? c[2] : c[3];
    const uint32_t r0 = __shfl_xor_sync(0xffffffffu, s0, 1), r1 = __shfl_xor_sync(0xffffffffu, s1, 1);
    if (b0) { c[0] = r0; c[2] = r1; } else { c[1] = r0; c[3] = r1; }
  }
}

// word (8 elements as 4 x bf16x2) -> 32 bytes of fp32 or 16 bytes of bf16 at dst
template <int OUT_BF16>
__device__ __forceinline__ void store_word(uint8_t* dst, const uint32_t* pr, bool wide) {
  if (OUT_BF16) {
    *reinterpret_cast<uint4*>(dst) = make_uint4(pr[0], pr[1], pr[2], pr[3]);
  } else {
    uint32_t v[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      v[2 * j] = pr[j] << 16;
      v[2 * j + 1] = pr[j] & 0xffff0000u;
    }
    store_b32x8(dst, v, wide);
  }
}

// Flat decode for 32-element blocks without residuals.  A lane loads the 16 code bytes and the
// metadata of one block (one 128-bit and one 16-bit load); the quad transposes the code words so
// that lane p decodes word p of the quad's four blocks and the quad stores contiguous lines.
// kDecodeUnroll blocks per thread are in flight; the loads of the next step are issued before the
// current step is decoded.
template <int OUT_BF16>
__global__ void __launch_bounds__(kDecodeThreads)
fb4_dequantize_b32_kernel(const uint32_t* __restrict__ codes, const uint16_t* __restrict__ meta, int64_t total_blocks,
                          const Fb4DeviceTables* __restrict__ tables, void* __restrict__ out, int out_aligned32) {
  __shared__ uint4 fb_bf16[32];   // per dialect: high bytes (8) then low bytes (8) of its magnitudes as bf16
  {
    const uint32_t bits = __float_as_uint((float)tables->formatbook[threadIdx.x >> 3][threadIdx.x & 7]) >> 16;
    uint8_t* row = reinterpret_cast<uint8_t*>(&fb_bf16[threadIdx.x >> 3]);
    row[threadIdx.x & 7] = (uint8_t)(bits >> 8);
    row[8 + (threadIdx.x & 7)] = (uint8_t)bits;
  }
  __syncthreads();
  const bool wide = out_aligned32 != 0;
  const int lane = threadIdx.x & 31;
  const int qp = lane & 3;
  constexpr int kWordBytes = OUT_BF16 ? 16 : 32;
  constexpr int64_t kStep = (int64_t)kDecodeThreads * kDecodeUnroll;
  const int64_t stride = (int64_t)gridDim.x * kStep;

  uint32_t cw[kDecodeUnroll][4], m[kDecodeUnroll];
  auto load = [&](int64_t base) {
#pragma unroll
    for (int u = 0; u < kDecodeUnroll; ++u) {
      const int64_t b = base + u * kDecodeThreads + threadIdx.x;
      cw[u][0] = cw[u][1] = cw[u][2] = cw[u][3] = 0u;
      m[u] = 0u;
      if (b < total_blocks) {
        load_block_codes<4>(codes + b * 4, cw[u]);
        m[u] = (uint32_t)__ldg(meta + b);
      }
    }
  };
  int64_t base = (int64_t)blockIdx.x * kStep;
  if (base < total_blocks) load(base);
  for (; base < total_blocks; base += stride) {
    uint32_t c[kDecodeUnroll][4], mm[kDecodeUnroll];
#pragma unroll
    for (int u = 0; u < kDecodeUnroll; ++u) {
      mm[u] = m[u];
#pragma unroll
      for (int k = 0; k < 4; ++k) c[u][k] = cw[u][k];
    }
    if (base + stride < total_blocks) load(base + stride);
#pragma unroll
    for (int u = 0; u < kDecodeUnroll; ++u) {
      quad_transpose(c[u], lane);
      const int64_t qb = base + u * kDecodeThreads + (threadIdx.x & ~3);   // first block of this quad
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t mi = __shfl_sync(0xffffffffu, mm[u], (lane & ~3) + i);
        if (qb + i < total_blocks) {
          uint32_t pr[4];
          decode_word(c[u][i], fb_bf16[(mi >> 8) & 31u], scale_bf16x2(mi), pr);
          store_word<OUT_BF16>(reinterpret_cast<uint8_t*>(out) + ((qb + i) * 4 + qp) * kWordBytes, pr, wide);
        }
      }
    }
  }
}

// Flat decode, general form: thread <-> one block (WPB code words of 8 elements, one metadata
// record); block size 16, and rows that add their decoded residual.  A thread keeps kDecodeUnroll
// blocks in flight, a CTA covers kDecodeThreads * kDecodeUnroll consecutive blocks per step, the
// grid strides.  codes and out are contiguous [T][C].
// RESID: rows listed in salient_idx (ascending) add their decoded residual (binary search per block).
template <int OUT_BF16, bool RESID, int WPB>
__global__ void __launch_bounds__(kDecodeThreads)
fb4_dequantize_kernel(const uint32_t* __restrict__ codes, const uint16_t* __restrict__ meta, int64_t total_blocks,
                      uint32_t blocks_per_row, const Fb4DeviceTables* __restrict__ tables,
                      const int32_t* __restrict__ salient_idx, int32_t n_salient,
                      const uint32_t* __restrict__ res_codes, const uint16_t* __restrict__ res_meta,
                      void* __restrict__ out, int out_aligned32) {
  __shared__ uint4 fb_bf16[32];   // per dialect: high bytes (8) then low bytes (8) of its magnitudes as bf16
  if (threadIdx.x < 256) {
    const uint32_t bits = __float_as_uint((float)tables->formatbook[threadIdx.x >> 3][threadIdx.x & 7]) >> 16;
    uint8_t* row = reinterpret_cast<uint8_t*>(&fb_bf16[threadIdx.x >> 3]);
    row[threadIdx.x & 7] = (uint8_t)(bits >> 8);
    row[8 + (threadIdx.x & 7)] = (uint8_t)bits;
  }
  __syncthreads();
  const bool wide = out_aligned32 != 0;
  constexpr int64_t kStep = (int64_t)kDecodeThreads * kDecodeUnroll;
  for (int64_t base = (int64_t)blockIdx.x * kStep; base < total_blocks; base += (int64_t)gridDim.x * kStep) {
    uint32_t cw[kDecodeUnroll][WPB], m[kDecodeUnroll];
#pragma unroll
    for (int u = 0; u < kDecodeUnroll; ++u) {
      const int64_t b = base + u * kDecodeThreads + threadIdx.x;
      if (b < total_blocks) {
        load_block_codes<WPB>(codes + b * WPB, cw[u]);
        m[u] = (uint32_t)__ldg(meta + b);
      }
    }
#pragma unroll
    for (int u = 0; u < kDecodeUnroll; ++u) {
      const int64_t b = base + u * kDecodeThreads + threadIdx.x;
      if (b >= total_blocks) continue;
      uint32_t pr[WPB * 4];   // two bf16 per register
      {
        const uint4 dt = fb_bf16[(m[u] >> 8) & 31u];
        const uint32_t sc2 = scale_bf16x2(m[u]);
#pragma unroll
        for (int k = 0; k < WPB; ++k) decode_word(cw[u][k], dt, sc2, pr + 4 * k);
      }
      int32_t srow = -1;
      int64_t rb = 0;
      if (RESID) {
        const int64_t t = b / blocks_per_row;
        int32_t lo = 0, hi = n_salient - 1;
        while (lo <= hi) {
          const int32_t mid = (lo + hi) >> 1;
          const int32_t sv = __ldg(salient_idx + mid);
          if (sv == (int32_t)t) { srow = mid; break; }
          if (sv < (int32_t)t) lo = mid + 1; else hi = mid - 1;
        }
        rb = (int64_t)srow * blocks_per_row + (b - t * blocks_per_row);
      }
      if (RESID && srow >= 0) {
        // Q(Act) + Q(Delta), rounded once to fp32 (Sec. 3.3)
        uint32_t rcw[WPB], rr[WPB * 4];
        load_block_codes<WPB>(res_codes + rb * WPB, rcw);
        const uint32_t rm = (uint32_t)__ldg(res_meta + rb);
        const uint4 rdt = fb_bf16[(rm >> 8) & 31u];
        const uint32_t rsc2 = scale_bf16x2(rm);
#pragma unroll
        for (int k = 0; k < WPB; ++k) decode_word(rcw[k], rdt, rsc2, rr + 4 * k);
        float v[WPB * 8];
#pragma unroll
        for (int j = 0; j < WPB * 4; ++j) {
          v[2 * j] = __fadd_rn(__uint_as_float(pr[j] << 16), __uint_as_float(rr[j] << 16));
          v[2 * j + 1] = __fadd_rn(__uint_as_float(pr[j] & 0xffff0000u), __uint_as_float(rr[j] & 0xffff0000u));
        }
        if (OUT_BF16) {
          uint32_t o[WPB * 4];
#pragma unroll
          for (int j = 0; j < WPB * 4; ++j) o[j] = f32_to_bf16_rne(v[2 * j]) | (f32_to_bf16_rne(v[2 * j + 1]) << 16);
          uint8_t* dst = reinterpret_cast<uint8_t*>(out) + b * (WPB * 16);
#pragma unroll
          for (int k = 0; k < WPB / 2; ++k) store_b32x8(dst + 32 * k, o + 8 * k, wide);
        } else {
          uint8_t* dst = reinterpret_cast<uint8_t*>(out) + b * (WPB * 32);
#pragma unroll
          for (int k = 0; k < WPB; ++k) store_b32x8(dst + 32 * k, reinterpret_cast<const uint32_t*>(v) + 8 * k, wide);
        }
      } else if (OUT_BF16) {
        uint8_t* dst = reinterpret_cast<uint8_t*>(out) + b * (WPB * 16);
#pragma unroll
        for (int k = 0; k < WPB / 2; ++k) store_b32x8(dst + 32 * k, pr + 8 * k, wide);
      } else {
        uint8_t* dst = reinterpret_cast<uint8_t*>(out) + b * (WPB * 32);
#pragma unroll
        for (int k = 0; k < WPB; ++k) store_word<0>(dst + 32 * k, pr + 4 * k, wide);
      }
    }
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
  const int B = (int)ctx->cfg.block_size;
  const int64_t blocks_per_row = C / B;
  if (blocks_per_row > 0x7fffffffLL || n_salient > 0x7fffffffLL) return cudaErrorInvalidValue;
  const int64_t total = T * blocks_per_row;
  constexpr int64_t kStep = (int64_t)kDecodeThreads * kDecodeUnroll;
  const int64_t want = (total + kStep - 1) / kStep;
  const int64_t cap = (int64_t)ctx->sm_count * 8;          // up to 8 CTAs of 256 threads per SM
  const unsigned grid = (unsigned)(want < cap ? want : cap);
  const uint32_t* cw = reinterpret_cast<const uint32_t*>(codes);
  const uint32_t* rw = reinterpret_cast<const uint32_t*>(res_codes);
  const int a32 = (reinterpret_cast<uintptr_t>(out) & 31u) == 0 ? 1 : 0;
#define FB4_DECODE(BF, RS, WPB)                                                                              \
  fb4_dequantize_kernel<BF, RS, WPB><<<grid, kDecodeThreads, 0, stream>>>(                                   \
      cw, meta, total, (uint32_t)blocks_per_row, ctx->d_tables, salient_idx, (int32_t)n_salient, rw, res_meta, out, a32)
#define FB4_DECODE_B(BF, RS)                          \
  do {                                                \
    if (B == 32) FB4_DECODE(BF, RS, 4); else FB4_DECODE(BF, RS, 2); \
  } while (0)
  if (n_salient == 0 && B == 32) {
    if (out_dtype == 1)
      fb4_dequantize_b32_kernel<1><<<grid, kDecodeThreads, 0, stream>>>(cw, meta, total, ctx->d_tables, out, a32);
    else
      fb4_dequantize_b32_kernel<0><<<grid, kDecodeThreads, 0, stream>>>(cw, meta, total, ctx->d_tables, out, a32);
  } else if (out_dtype == 1) {
    if (n_salient > 0) FB4_DECODE_B(1, true); else FB4_DECODE_B(1, false);
  } else {
    if (n_salient > 0) FB4_DECODE_B(0, true); else FB4_DECODE_B(0, false);
  }
#undef FB4_DECODE_B
#undef FB4_DECODE
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
