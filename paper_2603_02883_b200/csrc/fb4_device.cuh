// Device helpers shared by the kernels of libfb4 (decode of code words in registers).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace fb4dev {

// prmt.b32 in its default mode: selector bit 3 of a nibble replicates the sign of the chosen byte
// (the __byte_perm intrinsic only honours the low three bits).
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

__device__ __forceinline__ uint32_t mul_bf16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}

__device__ __forceinline__ float pow2f(int k) {   // 2^k, k in [-149,127]
  return k >= -126 ? __int_as_float((k + 127) << 23) : __int_as_float(1 << (k + 149));
}

// Entry d of the per-dialect magnitude table used by decode_word: the dialect's 8 magnitudes as
// bf16 bit patterns, high bytes in bytes 0..7, low bytes in bytes 8..15.  Thread i of 256 fills
// byte pair i (dialect i / 8, magnitude i % 8).
__device__ __forceinline__ void fill_fb_bf16(uint4* table, const uint8_t* formatbook /*[32][8]*/, int i) {
  const uint32_t bits = __float_as_uint((float)formatbook[i]) >> 16;   // integers 0..15 are exact in bf16
  uint8_t* row = reinterpret_cast<uint8_t*>(&table[i >> 3]);
  row[i & 7] = (uint8_t)(bits >> 8);
  row[8 + (i & 7)] = (uint8_t)bits;
}

// block scale 2^(sb-127), sb = low byte of the metadata record, as two bf16: sb << 7, or the
// subnormal 2^-127 = 0x0040 for sb = 0
__device__ __forceinline__ uint32_t scale_bf16x2(uint32_t m) {
  const uint32_t sb = m & 0xffu;
  return (sb ? (sb << 7) : 0x40u) * 0x10001u;
}

// One code word (8 elements) -> 4 registers of two bf16 values each (element 2j in the low half).
// dt = the dialect's entry of the magnitude table: a byte permute with the four 3-bit indices as
// selector looks up four magnitudes at once, no memory access per element.  One packed multiply
// applies the scale sc2.  Exact: a magnitude 0..15 times a power of two >= 2^-127 is a bf16
// value (subnormals included).
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

// e4m3 byte (1 sign, 4 exponent bits with bias 7, 3 mantissa bits) of an integer 0..15: exact
__host__ __device__ inline uint32_t e4m3_of_small_int(uint32_t m) {
  if (m == 0) return 0u;
  int ex = 0;
  while ((m >> (ex + 1)) != 0) ++ex;   // floor(log2 m) <= 3
  const uint32_t frac = m - (1u << ex);
  return ((uint32_t)(ex + 7) << 3) | (frac << 3 >> ex);
}

// 8 codes (one 32-bit code word) -> 8 e4m3 bytes (two registers).  fb = the dialect's 8 magnitudes as
// e4m3 bytes: a byte permute with four 3-bit indices as selector looks up four elements at once;
// sign bits come from sign-replicating permutes.
__device__ __forceinline__ void codes_to_e4m3(uint32_t cw, uint2 fb, uint32_t& lo, uint32_t& hi) {
  const uint32_t sel = cw & 0x77777777u;
  const uint32_t s_odd = prmt(cw, 0u, 0xba98u), s_even = prmt(cw << 4, 0u, 0xba98u);   // 0xff where negative
  lo = prmt(fb.x, fb.y, sel) | (__byte_perm(s_even, s_odd, 0x5140) & 0x80808080u);
  hi = prmt(fb.x, fb.y, sel >> 16) | (__byte_perm(s_even, s_odd, 0x7362) & 0x80808080u);
}

// Byte offset of the E8M0 scale of (row, 32-element block col): row-major, or tiles of 128 rows x 4
// columns (512 bytes, column tiles contiguous, (r mod 32)*16 + (r div 32)*4 + c inside a tile).
__host__ __device__ inline int64_t mx_scale_offset(int64_t row, int64_t col, int64_t n_col, int64_t col_tiles,
                                                   int tiled) {
  if (!tiled) return row * n_col + col;
  const int64_t r = row & 127;
  return ((row >> 7) * col_tiles + (col >> 2)) * 512 + (r & 31) * 16 + (r >> 5) * 4 + (col & 3);
}

}  // namespace fb4dev
