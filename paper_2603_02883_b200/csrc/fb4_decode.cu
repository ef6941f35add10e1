// FB4 decode (4-bit codes + block metadata -> fp32 / bf16, optionally adding the decoded
// residual of salient tokens) and the per-tile salient-token selection.
#include "fb4_block.cuh"
#include "fb4_device.cuh"
#include "fb4_internal.h"

namespace {

using fb4dev::decode_word;
using fb4dev::scale_bf16x2;

constexpr int kDecodeThreads = 256;
constexpr int kDecodeUnroll = 4;          // blocks in flight per thread

// two fp32 -> two bf16 (round to nearest even), low half = a
__device__ __forceinline__ uint32_t f32x2_to_bf16x2(float a, float b) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(b), "f"(a));
  return d;
}

// two fp32 -> two IEEE halves (round to nearest even, overflow to infinity), low half = a
__device__ __forceinline__ uint32_t f32x2_to_f16x2(float a, float b) {
  uint32_t d;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(b), "f"(a));
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

// word (8 elements as 4 x bf16x2) -> 32 bytes of fp32 (OUT 0), 16 bytes of bf16 (1) or of IEEE half (2) at dst
template <int OUT>
__device__ __forceinline__ void store_word(uint8_t* dst, const uint32_t* pr, bool wide) {
  if (OUT == 1) {
    *reinterpret_cast<uint4*>(dst) = make_uint4(pr[0], pr[1], pr[2], pr[3]);
  } else if (OUT == 2) {
    uint32_t h[4];
#pragma unroll
    for (int j = 0; j < 4; ++j)
      h[j] = f32x2_to_f16x2(__uint_as_float(pr[j] << 16), __uint_as_float(pr[j] & 0xffff0000u));
    *reinterpret_cast<uint4*>(dst) = make_uint4(h[0], h[1], h[2], h[3]);
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

// Sum of a decoded word and a decoded residual word (8 elements each as 4 x bf16x2), rounded once to
// fp32, then stored as fp32 / bf16 / half at dst.
template <int OUT_BF16>
__device__ __forceinline__ void store_sum_word(uint8_t* dst, const uint32_t* pr, const uint32_t* rr, bool wide) {
  uint32_t v[8];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    // float32 sums by the mixed-precision add (the bf16 halves are read where they lie: two operations on the
    // FMA pipe per element instead of two unpacking operations on the ALU pipe and an add)
    v[2 * j] = __float_as_uint(fb4blk::bf16_plus_f32<0>(pr[j], fb4blk::bf16_plus_f32<0>(rr[j], -0.0f)));
    v[2 * j + 1] = __float_as_uint(fb4blk::bf16_plus_f32<1>(pr[j], fb4blk::bf16_plus_f32<1>(rr[j], -0.0f)));
  }
  if (OUT_BF16 == 1) {
    uint4 o;
    o.x = f32x2_to_bf16x2(__uint_as_float(v[0]), __uint_as_float(v[1]));
    o.y = f32x2_to_bf16x2(__uint_as_float(v[2]), __uint_as_float(v[3]));
    o.z = f32x2_to_bf16x2(__uint_as_float(v[4]), __uint_as_float(v[5]));
    o.w = f32x2_to_bf16x2(__uint_as_float(v[6]), __uint_as_float(v[7]));
    *reinterpret_cast<uint4*>(dst) = o;
  } else if (OUT_BF16 == 2) {
    uint4 o;
    o.x = f32x2_to_f16x2(__uint_as_float(v[0]), __uint_as_float(v[1]));
    o.y = f32x2_to_f16x2(__uint_as_float(v[2]), __uint_as_float(v[3]));
    o.z = f32x2_to_f16x2(__uint_as_float(v[4]), __uint_as_float(v[5]));
    o.w = f32x2_to_f16x2(__uint_as_float(v[6]), __uint_as_float(v[7]));
    *reinterpret_cast<uint4*>(dst) = o;
  } else {
    store_b32x8(dst, v, wide);
  }
}

// Rows at least this wide (in 32-element units) get their residual added inside the flat decode.
// A step of 1024 units then spans at most 5 rows, so most steps hold no salient token and run the
// plain code; with narrower rows most steps would take the slower branch (at 96 units per row the
// fused kernel took 85 us against 81 us for the two kernels, fp32 output, and 70 against 49 us, bf16).
// The 16-bit outputs keep the two kernels at every width: their plain steps are short, the branch
// with the residual is not (75600 x 12288: bf16 0.396 against 0.402 ms, half 0.402 against 0.427 ms).
constexpr int64_t kFusedResidualMinUnitsPerRow = 256;

// The residual tensor of salient rows, for the flat decode that adds it in the same pass
struct ResidualRows {
  const int32_t* salient_idx;   // ascending token ids
  int64_t n_salient;
  const uint32_t* res_codes;    // [n_salient][units_per_row * 4 words]
  const uint16_t* res_meta;     // [n_salient][units_per_row]
  uint32_t units_per_row;
  float guess_scale;            // n_salient / T: list position of a row, to first order
  int64_t T;
  uint32_t* status;
};

// Flat decode without residuals, in units of 32 elements (one block of 32, or two blocks of 16).
// A lane loads the 16 code bytes of one unit (one 128-bit load) and the metadata records of its
// whole quad (one 64- or 128-bit load); the quad transposes the code words so that lane p decodes
// word p of the quad's four units and the quad stores contiguous lines.  kDecodeUnroll units per
// thread are in flight; the loads of the next step are issued before the current step is decoded.
// RESID (block size 32, fewer than 2^32 units): rows listed in rr.salient_idx also get their decoded
// residual added (Sec. 3.3: Q(Act) + Q(Delta), rounded once to fp32) in the same pass.  Per step the
// CTA finds the first list entry at or after the step's first row; a step whose rows hold no
// salient token (most of them) runs the plain code, the others look up each unit's row, load the
// residual codes of salient rows and add.
template <int OUT_BF16, bool B16, bool RESID, int UNROLL = kDecodeUnroll>
__global__ void __launch_bounds__(kDecodeThreads, 3)
fb4_dequantize_b32_kernel(const uint32_t* __restrict__ codes, const uint16_t* __restrict__ meta, int64_t total_units,
                          const Fb4DeviceTables* __restrict__ tables, void* __restrict__ out, int out_aligned32,
                          ResidualRows rr) {
  __shared__ uint4 fb_bf16[32];   // per dialect: high bytes (8) then low bytes (8) of its magnitudes as bf16
  fb4dev::fill_fb_bf16(fb_bf16, &tables->formatbook[0][0], threadIdx.x);
  __syncthreads();
  const bool wide = out_aligned32 != 0;
  const int lane = threadIdx.x & 31;
  const int qp = lane & 3;
  constexpr int RPU = B16 ? 2 : 1;   // metadata records per unit
  constexpr int kWordBytes = OUT_BF16 ? 16 : 32;
  constexpr int64_t kStep = (int64_t)kDecodeThreads * UNROLL;
  int64_t base = (int64_t)blockIdx.x * kStep, end = total_units, stride = (int64_t)gridDim.x * kStep;
  int64_t pos = 0;   // RESID: first list entry at or after the current step's first row
  if (RESID && blockIdx.x == 0) {   // entries outside the tensor match no row; they are reported
    bool bad = false;
    for (int64_t i = threadIdx.x; i < rr.n_salient; i += kDecodeThreads) {
      const int32_t r = __ldg(rr.salient_idx + i);
      bad |= r < 0 || r >= rr.T;
    }
    if (bad) atomicOr(rr.status, 2u);
  }

  // m = the metadata records of the lane's whole quad (4 units): after the transpose a lane decodes
  // one word of each of the quad's units and needs the record that covers it
  uint32_t cw[UNROLL][4];
  uint32_t m[UNROLL][2 * RPU];
  auto load = [&](int64_t base) {
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int64_t b = base + u * kDecodeThreads + threadIdx.x;
      const int64_t qb = b & ~3ll;
      cw[u][0] = cw[u][1] = cw[u][2] = cw[u][3] = 0u;
#pragma unroll
      for (int k = 0; k < 2 * RPU; ++k) m[u][k] = 0u;
      if (b < total_units) load_block_codes<4>(codes + b * 4, cw[u]);
      if (qb + 4 <= total_units) {   // aligned: qb is a multiple of 4
        if (B16) {
          const uint4 v = __ldg(reinterpret_cast<const uint4*>(meta + qb * 2));
          m[u][0] = v.x; m[u][1] = v.y; m[u][2 % (2 * RPU)] = v.z; m[u][3 % (2 * RPU)] = v.w;
        } else {
          const uint2 v = __ldg(reinterpret_cast<const uint2*>(meta + qb));
          m[u][0] = v.x; m[u][1] = v.y;
        }
      } else if (qb < total_units) {   // ragged last quad
        for (int i = 0; i < 4 * RPU; ++i)
          if (qb * RPU + i < total_units * RPU)
            m[u][i >> 1] |= (uint32_t)__ldg(meta + qb * RPU + i) << (16 * (i & 1));
      }
    }
  };
  if (base < end) load(base);
  for (; base < end; base += stride) {
    uint32_t c[UNROLL][4], mm[UNROLL][2 * RPU];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
#pragma unroll
      for (int k = 0; k < 2 * RPU; ++k) mm[u][k] = m[u][k];
#pragma unroll
      for (int k = 0; k < 4; ++k) c[u][k] = cw[u][k];
    }
    if (base + stride < end) load(base + stride);
    if (RESID) {
      // rows of this step: [row_first, row_last]; uniform over the CTA
      const uint32_t last_unit = (uint32_t)(base + kStep < total_units ? base + kStep : total_units) - 1u;
      const int64_t row_first = (uint32_t)base / rr.units_per_row, row_last = last_unit / rr.units_per_row;
      {
        // lower bound of row_first in the ascending list.  Salient tokens are spread over the sequence
        // (one per tile of tokens), so the entry sits next to the proportional guess: a few probes
        // around it, else a binary search.
        int64_t g = (int64_t)((float)row_first * rr.guess_scale);
        g = g < 0 ? 0 : (g > rr.n_salient ? rr.n_salient : g);
        int tries = 0;
        while (g > 0 && (int64_t)__ldg(rr.salient_idx + g - 1) >= row_first && tries < 8) { --g; ++tries; }
        while (g < rr.n_salient && (int64_t)__ldg(rr.salient_idx + g) < row_first && tries < 8) { ++g; ++tries; }
        if (tries == 8) {
          int64_t lo = 0, hi = rr.n_salient;
          while (lo < hi) {
            const int64_t mid = (lo + hi) >> 1;
            if ((int64_t)__ldg(rr.salient_idx + mid) < row_first) lo = mid + 1; else hi = mid;
          }
          g = lo;
        }
        pos = g;
      }
      const int64_t r0 = pos < rr.n_salient ? (int64_t)__ldg(rr.salient_idx + pos) : row_last + 1;
      if (r0 <= row_last) {
        // a salient row in this step.  Per warp and unit slot: the lanes look up their unit's row; if
        // none of the 32 units lies in a salient row the plain code runs, else the lanes of salient
        // rows load their residual codes and the quad adds the decoded residual.
        const bool more = pos + 1 < rr.n_salient && (int64_t)__ldg(rr.salient_idx + pos + 1) <= row_last;
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
          const int64_t b = base + u * kDecodeThreads + threadIdx.x;
          int64_t s = -1;              // residual row of this lane's unit
          uint32_t col = 0;
          if (b < total_units) {
            const uint32_t row = (uint32_t)b / rr.units_per_row;
            col = (uint32_t)b - row * rr.units_per_row;
            if ((int64_t)row == r0) {
              s = pos;
            } else if (more && (int64_t)row > r0) {
              for (int64_t k = pos + 1; k < rr.n_salient; ++k) {
                const int64_t r = (int64_t)__ldg(rr.salient_idx + k);
                if (r >= (int64_t)row) {
                  if (r == (int64_t)row) s = k;
                  break;
                }
              }
            }
          }
          const bool any_res = __any_sync(0xffffffffu, s >= 0);
          quad_transpose(c[u], lane);
          const int64_t qb = base + u * kDecodeThreads + (threadIdx.x & ~3);
          if (!any_res) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const uint32_t mi = (mm[u][i >> 1] >> (16 * (i & 1))) & 0xffffu;
              if (qb + i < total_units) {
                uint32_t pr[4];
                decode_word(c[u][i], fb_bf16[(mi >> 8) & 31u], scale_bf16x2(mi), pr);
                store_word<OUT_BF16>(reinterpret_cast<uint8_t*>(out) + ((qb + i) * 4 + qp) * kWordBytes, pr, wide);
              }
            }
            continue;
          }
          uint32_t rcw[4] = {0u, 0u, 0u, 0u}, rm = 0u;
          if (s >= 0) {
            load_block_codes<4>(rr.res_codes + (s * rr.units_per_row + col) * 4, rcw);
            rm = (uint32_t)__ldg(rr.res_meta + s * rr.units_per_row + col);
          }
          quad_transpose(rcw, lane);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int src = (lane & ~3) + i;
            const uint32_t mi = (mm[u][i >> 1] >> (16 * (i & 1))) & 0xffffu;
            const uint32_t rmi = __shfl_sync(0xffffffffu, rm, src);
            const bool has_res = __shfl_sync(0xffffffffu, (int)(s >= 0), src) != 0;
            if (qb + i < total_units) {
              uint32_t pr[4];
              decode_word(c[u][i], fb_bf16[(mi >> 8) & 31u], scale_bf16x2(mi), pr);
              uint8_t* dst = reinterpret_cast<uint8_t*>(out) + ((qb + i) * 4 + qp) * kWordBytes;
              if (has_res) {
                uint32_t rd[4];
                decode_word(rcw[i], fb_bf16[(rmi >> 8) & 31u], scale_bf16x2(rmi), rd);
                store_sum_word<OUT_BF16>(dst, pr, rd, wide);
              } else {
                store_word<OUT_BF16>(dst, pr, wide);
              }
            }
          }
        }
        continue;
      }
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      quad_transpose(c[u], lane);
      const int64_t qb = base + u * kDecodeThreads + (threadIdx.x & ~3);   // first unit of this quad
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        // record of unit i (block 32), or of the half of unit i that holds word qp (block 16)
        const uint32_t mi = B16 ? (mm[u][i] >> (16 * (qp >> 1))) & 0xffffu
                                : (mm[u][i >> 1] >> (16 * (i & 1))) & 0xffffu;
        if (qb + i < total_units) {
          uint32_t pr[4];
          decode_word(c[u][i], fb_bf16[(mi >> 8) & 31u], scale_bf16x2(mi), pr);
          store_word<OUT_BF16>(reinterpret_cast<uint8_t*>(out) + ((qb + i) * 4 + qp) * kWordBytes, pr, wide);
        }
      }
    }
  }
}

// Flat decode, general form (block size 16): thread <-> one block (WPB code words of 8 elements,
// one metadata record).  A thread keeps kDecodeUnroll blocks in flight, a CTA covers
// kDecodeThreads * kDecodeUnroll consecutive blocks per step, the grid strides.
template <int OUT_BF16, int WPB>
__global__ void __launch_bounds__(kDecodeThreads)
fb4_dequantize_kernel(const uint32_t* __restrict__ codes, const uint16_t* __restrict__ meta, int64_t total_blocks,
                      const Fb4DeviceTables* __restrict__ tables, void* __restrict__ out, int out_aligned32) {
  __shared__ uint4 fb_bf16[32];   // per dialect: high bytes (8) then low bytes (8) of its magnitudes as bf16
  fb4dev::fill_fb_bf16(fb_bf16, &tables->formatbook[0][0], threadIdx.x);
  __syncthreads();
  const bool wide = out_aligned32 != 0;
  constexpr int kWordBytes = OUT_BF16 ? 16 : 32;
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
      const uint4 dt = fb_bf16[(m[u] >> 8) & 31u];
      const uint32_t sc2 = scale_bf16x2(m[u]);
#pragma unroll
      for (int k = 0; k < WPB; ++k) {
        uint32_t pr[4];
        decode_word(cw[u][k], dt, sc2, pr);
        store_word<OUT_BF16>(reinterpret_cast<uint8_t*>(out) + (b * WPB + k) * kWordBytes, pr, wide);
      }
    }
  }
}

// Rows with a residual (Sec. 3.3: Q(Act) + Q(Delta), the sum rounded once to fp32): thread <-> one
// block of one salient row; decodes the main and the residual codes and writes the row of `out`
// again.  Runs after the flat decode on the same stream.  An entry of salient_idx outside [0, T) is
// skipped and raises bit 1 of the status word.  With 32-element blocks (WPB 4) the code
// words are transposed inside each quad of lanes, as in the flat kernel, so that a quad stores
// whole lines; block index and metadata of the quad's other blocks come by shuffle (a quad may
// straddle two salient rows, so each block keeps its own destination).
template <int OUT_BF16, int WPB>
__global__ void __launch_bounds__(kDecodeThreads)
fb4_dequantize_residual_rows_kernel(const uint32_t* __restrict__ codes, const uint16_t* __restrict__ meta,
                                    uint32_t blocks_per_row, const Fb4DeviceTables* __restrict__ tables,
                                    const int32_t* __restrict__ salient_idx, int64_t n_salient,
                                    const uint32_t* __restrict__ res_codes, const uint16_t* __restrict__ res_meta,
                                    void* __restrict__ out, int out_aligned32, int64_t T,
                                    uint32_t* __restrict__ status) {
  __shared__ uint4 fb_bf16[32];
  fb4dev::fill_fb_bf16(fb_bf16, &tables->formatbook[0][0], threadIdx.x);
  __syncthreads();
  const bool wide = out_aligned32 != 0;
  constexpr int kWordBytes = OUT_BF16 ? 16 : 32;
  const int64_t total = n_salient * blocks_per_row;
  const int lane = threadIdx.x & 31, qp = lane & 3;
  // the loop bound is warp-uniform (first lane's block), so that the shuffles below are convergent
  for (int64_t rb = (int64_t)blockIdx.x * kDecodeThreads + threadIdx.x; rb - lane < total;
       rb += (int64_t)gridDim.x * kDecodeThreads) {
    uint32_t cw[WPB], rcw[WPB], m = 0u, rm = 0u;
#pragma unroll
    for (int k = 0; k < WPB; ++k) cw[k] = rcw[k] = 0u;
    int64_t b = -1;   // destination block; -1 = past the end
    if (rb < total) {
      // 32-bit division whenever the block index fits (a 64-bit one costs about a hundred instructions)
      const int64_t srow = total <= 0xffffffffLL ? (int64_t)((uint32_t)rb / blocks_per_row) : rb / blocks_per_row;
      const int64_t row = (int64_t)__ldg(salient_idx + srow);
      if (row >= 0 && row < T) {
        b = row * blocks_per_row + (rb - srow * blocks_per_row);
        load_block_codes<WPB>(codes + b * WPB, cw);
        load_block_codes<WPB>(res_codes + rb * WPB, rcw);
        m = (uint32_t)__ldg(meta + b);
        rm = (uint32_t)__ldg(res_meta + rb);
      } else {
        atomicOr(status, 2u);   // a token index outside the tensor: the entry is skipped and reported
      }
    }
    if (WPB == 4) {
      uint32_t c4[4] = {cw[0], cw[1], cw[2 % WPB], cw[3 % WPB]};
      uint32_t r4[4] = {rcw[0], rcw[1], rcw[2 % WPB], rcw[3 % WPB]};
      quad_transpose(c4, lane);
      quad_transpose(r4, lane);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int src = (lane & ~3) + i;
        const uint32_t mi = __shfl_sync(0xffffffffu, m, src), rmi = __shfl_sync(0xffffffffu, rm, src);
        const int64_t bi = __shfl_sync(0xffffffffu, b, src);
        if (bi < 0) continue;
        uint32_t pr[4], rr[4];
        decode_word(c4[i], fb_bf16[(mi >> 8) & 31u], scale_bf16x2(mi), pr);
        decode_word(r4[i], fb_bf16[(rmi >> 8) & 31u], scale_bf16x2(rmi), rr);
        store_sum_word<OUT_BF16>(reinterpret_cast<uint8_t*>(out) + (bi * 4 + qp) * kWordBytes, pr, rr, wide);
      }
    } else {
      if (b < 0) continue;
      const uint4 dt = fb_bf16[(m >> 8) & 31u], rdt = fb_bf16[(rm >> 8) & 31u];
      const uint32_t sc2 = scale_bf16x2(m), rsc2 = scale_bf16x2(rm);
#pragma unroll
      for (int k = 0; k < WPB; ++k) {
        uint32_t pr[4], rr[4];
        decode_word(cw[k], dt, sc2, pr);
        decode_word(rcw[k], rdt, rsc2, rr);
        store_sum_word<OUT_BF16>(reinterpret_cast<uint8_t*>(out) + (b * WPB + k) * kWordBytes, pr, rr, wide);
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

// The k highest scores of the whole sequence (ties to the lowest index), indices in ascending order:
// the global reading of "top 5 % of the tokens".  One CTA: a 4-pass radix select finds the k-th
// largest key, then one ordered pass writes the indices above it and the first few equal to it.
constexpr int kTopkThreads = 1024;

__device__ __forceinline__ uint32_t score_key(float f) {   // order-preserving; -0 counts as +0
  uint32_t u = __float_as_uint(f);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__global__ void __launch_bounds__(kTopkThreads)
fb4_select_salient_topk_kernel(const float* __restrict__ score, int64_t T, int64_t k,
                               int32_t* __restrict__ salient_idx) {
  __shared__ uint32_t hist[256];
  __shared__ uint32_t s_prefix, s_remaining;
  __shared__ uint32_t warp_sums[kTopkThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { s_prefix = 0u; s_remaining = (uint32_t)k; }
  for (int pass = 3; pass >= 0; --pass) {
    if (tid < 256) hist[tid] = 0u;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const uint32_t high_mask = pass == 3 ? 0u : (0xffffffffu << (8 * (pass + 1)));
    for (int64_t t = tid; t < T; t += kTopkThreads) {
      const uint32_t key = score_key(score[t]);
      if ((key & high_mask) == prefix) atomicAdd(&hist[(key >> (8 * pass)) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {   // walk the bins from the top until the k-th largest key falls into one
      uint32_t remaining = s_remaining;
      int bin = 255;
      for (; bin > 0; --bin) {
        if (hist[bin] >= remaining) break;
        remaining -= hist[bin];
      }
      s_remaining = remaining;
      s_prefix = prefix | ((uint32_t)bin << (8 * pass));
    }
    __syncthreads();
  }
  const uint32_t kth = s_prefix;          // key of the k-th largest score
  const uint32_t quota = s_remaining;     // how many scores equal to it are taken (lowest indices first)
  uint32_t written = 0, ties_seen = 0;    // uniform across the CTA
  for (int64_t base = 0; base < T; base += kTopkThreads) {
    const int64_t t = base + tid;
    uint32_t g = 0, e = 0;
    if (t < T) {
      const uint32_t key = score_key(score[t]);
      g = key > kth;
      e = key == kth;
    }
    // exclusive counts of greater / equal elements before this thread within the chunk
    const uint32_t bg = __ballot_sync(0xffffffffu, g), be = __ballot_sync(0xffffffffu, e);
    const uint32_t lower = (1u << lane) - 1u;
    uint32_t gb = __popc(bg & lower), eb = __popc(be & lower);
    if (lane == 0) warp_sums[warp] = (__popc(bg) << 16) | __popc(be);
    __syncthreads();
    uint32_t before = 0, total = 0;
    for (int w = 0; w < kTopkThreads / 32; ++w) {
      const uint32_t v = warp_sums[w];
      if (w < warp) before += v;
      total += v;
    }
    __syncthreads();
    gb += before >> 16;
    eb += before & 0xffffu;
    const uint32_t quota_left = quota > ties_seen ? quota - ties_seen : 0u;
    if (g) salient_idx[written + gb + min(eb, quota_left)] = (int32_t)t;
    else if (e && eb < quota_left) salient_idx[written + gb + eb] = (int32_t)t;
    written += (total >> 16) + min(total & 0xffffu, quota_left);
    ties_seen += total & 0xffffu;
  }
}

}  // namespace

cudaError_t fb4_launch_dequantize(const fb4_ctx* ctx, const uint8_t* codes, const uint16_t* meta, int64_t T,
                                  int64_t C, const int32_t* salient_idx, int64_t n_salient,
                                  const uint8_t* res_codes, const uint16_t* res_meta, void* out, int out_dtype,
                                  cudaStream_t stream, int* launches) {
  static_assert(kDecodeThreads == 256, "one thread per formatbook entry fills the shared table");
  *launches = 0;
  if (T == 0 || C == 0) return cudaSuccess;
  const int B = (int)ctx->cfg.block_size;
  const int64_t blocks_per_row = C / B;
  if (blocks_per_row > 0x7fffffffLL) return cudaErrorInvalidValue;
  const int64_t total = T * blocks_per_row;
  constexpr int64_t kStep = (int64_t)kDecodeThreads * kDecodeUnroll;
  // One step per CTA, no persistent loop: with CTAs dispatched in order the whole GPU works on one
  // narrow, advancing window of the output, which the memory system takes better than a few hundred
  // resident CTAs streaming far apart (fp32 output: 0.695 -> 0.646 ms at 75600 x 12288).  The kernels
  // keep their grid-stride loops for the few shapes whose step count exceeds the grid limit.
  const int64_t cap = 0x7fffffff;
  const int64_t want = (total + kStep - 1) / kStep;
  const unsigned grid = (unsigned)(want < cap ? want : cap);
  const uint32_t* cw = reinterpret_cast<const uint32_t*>(codes);
  const uint32_t* rw = reinterpret_cast<const uint32_t*>(res_codes);
  const int a32 = (reinterpret_cast<uintptr_t>(out) & 31u) == 0 ? 1 : 0;
  const Fb4DeviceTables* tb = ctx->d_tables;
#define FB4_BY_DTYPE(CALL)          \
  do {                              \
    if (out_dtype == 1) { CALL(1); } \
    else if (out_dtype == 2) { CALL(2); } \
    else { CALL(0); }               \
  } while (0)
  ResidualRows none{};
  if (B == 32 && n_salient > 0 && blocks_per_row >= kFusedResidualMinUnitsPerRow && total < 0xffffffffLL &&
      out_dtype == 0) {   // fp32 output only: for the 16-bit outputs the two kernels measure faster
    // residual rows added in the same pass: every row is written once
    const ResidualRows rr{salient_idx, n_salient, rw, res_meta, (uint32_t)blocks_per_row,
                          (float)((double)n_salient / (double)T), T, ctx->d_status};
    fb4_dequantize_b32_kernel<0, false, true><<<grid, kDecodeThreads, 0, stream>>>(cw, meta, total, tb, out, a32, rr);
    const cudaError_t fe = cudaGetLastError();
    if (fe == cudaSuccess) *launches = 1;
    return fe;
  }
  if (B == 32 && want < (int64_t)ctx->sm_count * 2) {
    // small tensor: one unit per thread, so that the few units there are spread over all SMs
    const unsigned sgrid = (unsigned)((total + kDecodeThreads - 1) / kDecodeThreads);
#define FB4_CALL(O) \
  fb4_dequantize_b32_kernel<O, false, false, 1><<<sgrid, kDecodeThreads, 0, stream>>>(cw, meta, total, tb, out, a32, none)
    FB4_BY_DTYPE(FB4_CALL);
#undef FB4_CALL
  } else if (B == 32) {
#define FB4_CALL(O) \
  fb4_dequantize_b32_kernel<O, false, false><<<grid, kDecodeThreads, 0, stream>>>(cw, meta, total, tb, out, a32, none)
    FB4_BY_DTYPE(FB4_CALL);
#undef FB4_CALL
  } else if (C % 32 == 0) {   // block 16 in units of two blocks
    const int64_t units = total / 2;
    const int64_t uwant = (units + kStep - 1) / kStep;
    const unsigned ugrid = (unsigned)(uwant < cap ? uwant : cap);
#define FB4_CALL(O) \
  fb4_dequantize_b32_kernel<O, true, false><<<ugrid, kDecodeThreads, 0, stream>>>(cw, meta, units, tb, out, a32, none)
    FB4_BY_DTYPE(FB4_CALL);
#undef FB4_CALL
  } else {
#define FB4_CALL(O) fb4_dequantize_kernel<O, 2><<<grid, kDecodeThreads, 0, stream>>>(cw, meta, total, tb, out, a32)
    FB4_BY_DTYPE(FB4_CALL);
#undef FB4_CALL
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  *launches = 1;
  if (n_salient > 0) {
    const int64_t rtotal = n_salient * blocks_per_row;
    const int64_t rwant = (rtotal + kDecodeThreads - 1) / kDecodeThreads;
    const unsigned rgrid = (unsigned)(rwant < cap ? rwant : cap);
    const uint32_t bpr = (uint32_t)blocks_per_row;
#define FB4_RESID(BF, WPB)                                                                 \
  fb4_dequantize_residual_rows_kernel<BF, WPB><<<rgrid, kDecodeThreads, 0, stream>>>(      \
      cw, meta, bpr, tb, salient_idx, n_salient, rw, res_meta, out, a32, T, ctx->d_status)
    if (B == 32) {
#define FB4_CALL(O) FB4_RESID(O, 4)
      FB4_BY_DTYPE(FB4_CALL);
#undef FB4_CALL
    } else {
#define FB4_CALL(O) FB4_RESID(O, 2)
      FB4_BY_DTYPE(FB4_CALL);
#undef FB4_CALL
    }
#undef FB4_RESID
    e = cudaGetLastError();
    if (e == cudaSuccess) *launches = 2;
  }
#undef FB4_BY_DTYPE
  return e;
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

cudaError_t fb4_launch_select_salient_topk(const float* score, int64_t T, int64_t k, int32_t* salient_idx,
                                           cudaStream_t stream) {
  if (T == 0 || k == 0) return cudaSuccess;
  fb4_select_salient_topk_kernel<<<1, kTopkThreads, 0, stream>>>(score, T, k, salient_idx);
  return cudaGetLastError();
}
