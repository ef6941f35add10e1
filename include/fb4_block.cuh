/*
 * fb4_block.cuh -- the per-block FB4 routine of libfb4 as device code a producer kernel can include.
 *
 * Sec. 3.1-3.2 of SemanticDialect for ONE block held in registers: scale from the block maximum,
 * group-wise maxima, two-stage dialect selection with the error table, table quantization of every
 * element (optionally restricted to a SeDA sub-formatbook, Sec. 3.4).  App. D.2 runs the quantizer as
 * the tail of the operation in front of it; a kernel that still holds its fp32 results in registers
 * calls fb4blk::quantize_block_f32 on them and stores 16 bytes of codes and one metadata record per
 * block - the activation never reaches memory in 16 bits.  The kernels of the library are built on
 * the same routine (quantize_packed_block), so this file cannot drift from them.
 *
 * Use (one thread per block; CUDA C++ for sm_100a):
 *   host:    fb4_block_tables(ctx, &image, &bytes)            // device pointer to the table image
 *   kernel:  extern __shared__ __align__(16) unsigned char smem[];
 *            fb4blk::Tables* tb = reinterpret_cast<fb4blk::Tables*>(smem);     // sizeof(fb4blk::Tables) bytes
 *            fb4blk::copy_tables(tb, image);  __syncthreads();                   // all threads of the CTA
 *            fb4blk::Lane ln = fb4blk::lane_state(tb);
 *            uint32_t codes[4]; uint16_t meta;
 *            fb4blk::quantize_block_f32(x, 0xffffffffu, tb, ln, codes, &meta);      // float x[32]
 *   The image matches the context it came from (formatbook, stage-1 table); the routines here implement
 *   block size 32, num_groups 8, two-stage selection and the full exponent range, the library's
 *   default configuration.  Contexts whose tables do not fit the packed layout return no image.
 *
 * Output: codes[q] holds elements 8q .. 8q+7, element k in nibble k (sign << 3 | index); meta = scale
 * byte | dialect << 8, exactly the layout of fb4_quantize.
 */
#ifndef FB4_BLOCK_CUH_
#define FB4_BLOCK_CUH_

#include <cuda_runtime.h>
#include <stdint.h>

namespace fb4blk {

constexpr int kPairMul = 36;         // pair-table address = 36*bin_hi + bin_lo: spreads small bins over the banks
constexpr int kPairStride = 1148;    // 36*31 + 32 bytes per dialect; 287 words: one bank of rotation per dialect
constexpr int kMaxGroups = 8;        // distinct stage-1 groups the packed tables hold

// prmt.b32 in its default mode: selector bit 3 of a nibble replicates the sign of the chosen byte
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

// Compact tables, built at init (the part of the shared-memory image that is read as is).
struct FastTables {
  uint8_t qvalue[32][32];                // [dialect][bin] -> index of the nearest magnitude
  uint64_t qerr64[kMaxGroups][32];       // [group][bin] -> byte j = Qerror of candidate j (pad 31)
  uint8_t did_of[kMaxGroups][8];         // [group][candidate] -> dialect id
  uint8_t group_of_bin[32];              // [bin of block maximum] -> group
  uint32_t stage1[32];                   // [bin of block maximum] -> candidate mask
  uint8_t qerror[32][32];                // [dialect][bin], for masks that cut a group
  uint8_t fb[32][8];
  uint32_t n_groups;                     // stage-1 groups in use
  uint32_t pad_[3];
  uint4 did_lanes[kMaxGroups];           // [group] -> dialect ids of candidates (2,0), (3,1), (6,4), (7,5) in 16-bit lanes
};
static_assert(sizeof(FastTables) % 16 == 0, "copied with 16-byte accesses");

// The tables as they sit in shared memory.  The image is built once on the host at init, kept in
// global memory, and copied by every CTA with one bulk asynchronous copy.
struct Tables {
  // [group][bin][lane & 15] -> the 8 candidate errors: each lane of a half-warp has its own
  // 8-byte column, so the 64-bit loads of a warp never conflict
  uint64_t qerr_private[kMaxGroups][32][16];
  uint8_t pairlut[32 * kPairStride];     // [dialect][36*bin_hi + bin_lo] -> idx_lo | idx_hi<<4
  uint4 fb_bf16[32];                     // [dialect] -> magnitudes as bf16, high bytes then low bytes (residual pass)
  uint2 fb_e4m3[32];                     // [dialect] -> magnitudes as e4m3 bytes (MXFP8 output)
  FastTables c;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint32_t lds_u8(uint32_t addr) {
  uint32_t v;
  asm("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
// A byte load that a flag switches off: with ok == 0 nothing is read and dst keeps the value it came with.
__device__ __forceinline__ void lds_u8_if(uint32_t& dst, uint32_t addr, uint32_t ok) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t@p ld.shared.u8 %0, [%1];\n\t}" : "+r"(dst) : "r"(addr), "r"(ok));
}
__device__ __forceinline__ uint2 lds_v2(uint32_t addr) {
  uint2 v;
  asm("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}
// Float32 sum / difference with one bf16 half of a packed register as the first operand (HALF 0 = low, 1 = high):
// the half is converted exactly and the result rounded once, as for __fadd_rn / __fsub_rn on the unpacked
// value, but the instruction reads the half where it lies, without the shift or mask that unpacks it.
template <int HALF>
__device__ __forceinline__ float bf16_plus_f32(uint32_t w, float c) {
  float d;
  if (HALF == 0)
    asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tadd.rn.f32.bf16 %0, lo, %2;\n\t}" : "=f"(d) : "r"(w), "f"(c));
  else
    asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tadd.rn.f32.bf16 %0, hi, %2;\n\t}" : "=f"(d) : "r"(w), "f"(c));
  return d;
}
template <int HALF>
__device__ __forceinline__ float bf16_minus_f32(uint32_t w, float c) {
  float d;
  if (HALF == 0)
    asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tsub.rn.f32.bf16 %0, lo, %2;\n\t}" : "=f"(d) : "r"(w), "f"(c));
  else
    asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tsub.rn.f32.bf16 %0, hi, %2;\n\t}" : "=f"(d) : "r"(w), "f"(c));
  return d;
}
// The low bf16 of a packed register as float32 (x + -0 = x for every x): the FMA pipe instead of a shift on the
// busier ALU pipe.
__device__ __forceinline__ float bf16_lo_as_f32(uint32_t w) { return bf16_plus_f32<0>(w, -0.0f); }
__device__ __forceinline__ uint4 lds_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

// Score an arbitrary candidate mask over 8 group bins with the byte table (SeDA masks that
// cut a stage-1 group).  Ascending ids: ties keep the lowest.
__device__ __forceinline__ int select_general(uint32_t cand, const uint8_t* gb, const Tables* tb) {
  int best = 0, best_err = 0x7fffffff;
  for (uint32_t m = cand; m; m &= m - 1) {
    const int d = __ffs((int)m) - 1;
    int err = 0;
#pragma unroll
    for (int g = 0; g < 8; ++g) err += tb->c.qerror[d][gb[g]];
    if (err < best_err) { best_err = err; best = d; }
  }
  return best;
}

// Dialect selection of one block (Sec. 3.2 two-stage; Sec. 3.4 restriction).  gm = the 8 group
// maxima as fp32 magnitudes (mantissa bits below the bin resolution are truncated away),
// sG = 2^(3-e) * 2^-21, bmax = bin of the block maximum, qerr_lane = this lane's column of the
// packed error table.
template <bool SEDA>
__device__ __forceinline__ int choose_dialect(const float (&gm)[8], float sG, uint32_t bmax, uint32_t allowed,
                                              const Tables* tb, uint32_t qerr_lane) {
  const uint32_t grp = tb->c.group_of_bin[bmax];
  bool packed_path = true;
  uint32_t cand = 0;
  if (SEDA) {
    const uint32_t st1 = tb->c.stage1[bmax];
    cand = st1 & allowed;
    if (cand == 0) cand = allowed;
    packed_path = (cand == st1);
  }
  if (!SEDA || packed_path) {
    const uint32_t qb = qerr_lane + grp * 4096u;
    uint32_t lo = 0, hi = 0;
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      const uint32_t t = __float_as_uint(__fmaf_rz(gm[g], sG, 2.0f));
      const uint2 e = lds_v2((t << 7) + qb);   // 0x40000000 << 7 vanishes mod 2^32: 128 B per bin
      lo += e.x;
      hi += e.y;
    }
    // argmin over 8 byte sums, ties to the lowest candidate: keys (err << 3 | j) in 16-bit lanes
    const uint32_t k02 = (lo & 0x00ff00ffu) * 8u + 0x00020000u;
    const uint32_t k13 = ((lo >> 8) & 0x00ff00ffu) * 8u + 0x00030001u;
    const uint32_t k46 = (hi & 0x00ff00ffu) * 8u + 0x00060004u;
    const uint32_t k57 = ((hi >> 8) & 0x00ff00ffu) * 8u + 0x00070005u;
    const uint32_t km = __vminu2(__vminu2(k02, k13), __vminu2(k46, k57));
    const uint32_t key = min(km & 0xffffu, km >> 16);
    return tb->c.did_of[grp][key & 7u];
  }
  if (__popc(cand) == 1) return __ffs((int)cand) - 1;
  uint8_t gb[8];
#pragma unroll
  for (int g = 0; g < 8; ++g) gb[g] = (uint8_t)(__float_as_uint(__fmaf_rz(gm[g], sG, 2.0f)) & 31u);
  return select_general(cand, gb, tb);
}

// num_groups = block size (every element is its own group, the setting of the paper's Table 2 comparison):
// the error of a candidate is summed over the bins of all 32 elements.  a = the 16 packed magnitude registers.
// Byte sums would overflow (32 terms of up to 31), so every run of 8 elements is added in bytes and then
// widened into 16-bit lanes; the keys are formed from those.
template <bool SEDA>
__device__ __forceinline__ int choose_dialect_per_element(const uint32_t (&a)[16], float sG, uint32_t bmax, uint32_t allowed,
                                                          const Tables* tb, uint32_t qerr_lane) {
  const uint32_t grp = tb->c.group_of_bin[bmax];
  uint32_t cand = 0;
  bool packed_path = true;
  if (SEDA) {
    const uint32_t st1 = tb->c.stage1[bmax];
    cand = st1 & allowed;
    if (cand == 0) cand = allowed;
    packed_path = (cand == st1);
  }
  if (!SEDA || packed_path) {
    const uint32_t qb = qerr_lane + grp * 4096u;
    uint32_t s02 = 0, s13 = 0, s46 = 0, s57 = 0;      // candidates (2, 0), (3, 1), (6, 4), (7, 5) in 16-bit lanes
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint32_t lo = 0, hi = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t av = a[4 * q + j];
        const uint32_t t1 = __float_as_uint(__fmaf_rz(__uint_as_float(av), sG, 2.0f));         // upper element
        const uint32_t t0 = __float_as_uint(__fmaf_rz(bf16_lo_as_f32(av), sG, 2.0f));   // lower element
        const uint2 e0 = lds_v2((t0 << 7) + qb), e1 = lds_v2((t1 << 7) + qb);
        lo += e0.x + e1.x;
        hi += e0.y + e1.y;
      }
      s02 += lo & 0x00ff00ffu;
      s13 += (lo >> 8) & 0x00ff00ffu;
      s46 += hi & 0x00ff00ffu;
      s57 += (hi >> 8) & 0x00ff00ffu;
    }
    const uint32_t k02 = s02 * 8u + 0x00020000u, k13 = s13 * 8u + 0x00030001u;
    const uint32_t k46 = s46 * 8u + 0x00060004u, k57 = s57 * 8u + 0x00070005u;
    const uint32_t km = __vminu2(__vminu2(k02, k13), __vminu2(k46, k57));
    const uint32_t key = min(km & 0xffffu, km >> 16);
    return tb->c.did_of[grp][key & 7u];
  }
  if (__popc(cand) == 1) return __ffs((int)cand) - 1;
  // a mask that cuts the stage-1 group: every candidate scored with the byte table (ascending ids: ties keep the lowest)
  int best = 0, best_err = 0x7fffffff;
  for (uint32_t m = cand; m; m &= m - 1) {
    const int d = __ffs((int)m) - 1;
    int err = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const uint32_t b1 = __float_as_uint(__fmaf_rz(__uint_as_float(a[i]), sG, 2.0f)) & 31u;
      const uint32_t b0 = __float_as_uint(__fmaf_rz(__uint_as_float(a[i] << 16), sG, 2.0f)) & 31u;
      err += tb->c.qerror[d][b0] + tb->c.qerror[d][b1];
    }
    if (err < best_err) { best_err = err; best = d; }
  }
  return best;
}

// select_mode 1: no stage 1, every allowed dialect is scored on the 8 group maxima (the plain comparison of all
// dialects that Sec. 3.2 starts from, with the table criterion).  The packed words of all stage-1 groups are
// summed in turn and compared as (error << 5 | dialect id) keys in 16-bit lanes; the smallest key wins, so ties go
// to the lowest id.  A SeDA mask other than all-ones takes the byte table.
template <bool SEDA>
__device__ __forceinline__ int choose_dialect_all(const float (&gm)[8], float sG, uint32_t allowed, const Tables* tb,
                                                  uint32_t qerr_lane) {
  uint32_t t[8];
#pragma unroll
  for (int g = 0; g < 8; ++g) t[g] = __float_as_uint(__fmaf_rz(gm[g], sG, 2.0f));
  if (SEDA && allowed != 0xffffffffu) {
    uint8_t gb[8];
#pragma unroll
    for (int g = 0; g < 8; ++g) gb[g] = (uint8_t)(t[g] & 31u);
    return select_general(allowed, gb, tb);
  }
  // running minima of (error << 5 | dialect id) in 16-bit lanes: byte lanes (2, 0), (3, 1), (6, 4), (7, 5) of the sums
  uint32_t m02 = 0xffffffffu, m13 = 0xffffffffu, m46 = 0xffffffffu, m57 = 0xffffffffu;
  const uint32_t n_groups = tb->c.n_groups;
  uint32_t addr[8];
#pragma unroll
  for (int g = 0; g < 8; ++g) addr[g] = (t[g] << 7) + qerr_lane;
#pragma unroll
  for (int grp = 0; grp < kMaxGroups; ++grp) {
    if ((uint32_t)grp < n_groups) {
      uint32_t lo = 0, hi = 0;
#pragma unroll
      for (int g = 0; g < 8; ++g) {
        const uint2 e = lds_v2(addr[g] + (uint32_t)grp * 4096u);
        lo += e.x;
        hi += e.y;
      }
      const uint4 ids = tb->c.did_lanes[grp];      // the candidates' dialect ids in the same lanes (pads: 31)
      m02 = __vminu2(m02, (lo & 0x00ff00ffu) * 32u + ids.x);
      m13 = __vminu2(m13, ((lo >> 8) & 0x00ff00ffu) * 32u + ids.y);
      m46 = __vminu2(m46, (hi & 0x00ff00ffu) * 32u + ids.z);
      m57 = __vminu2(m57, ((hi >> 8) & 0x00ff00ffu) * 32u + ids.w);
    }
  }
  // a pad sums to 248 and carries id 31: it ties at worst with the real dialect 31, the same answer
  const uint32_t km = __vminu2(__vminu2(m02, m13), __vminu2(m46, m57));
  const uint32_t best = min(km & 0xffffu, km >> 16);
  return (int)(best & 31u);
}

// One lane's block(s) from 16 registers of two 16-bit values each - bf16 inputs, or any fp32 values cut
// to their upper 16 bits: the scale exponent, the bins of the 0.5-wide tables and the sign are all
// fixed by those bits (every bin boundary is a multiple of the cut's granularity), so the cut loses
// nothing.  Scale, group maxima, dialect selection, LUT quantization; block size 32, or (B16) two
// blocks of 16; CLAMP: clamped exponent range.  Out: the four code words, and per half the chosen
// dialect and the biased exponent.
// SEL: 0 = 8 groups, two-stage selection (the default); 1 = every element its own group (block size 32 only);
// 2 = 8 groups, every allowed dialect scored (select_mode 1).
template <bool SEDA, bool B16, bool CLAMP, int SEL = 0, bool BRANCHY = false>
__device__ __forceinline__ void quantize_packed_block(const uint32_t (&w)[16], uint32_t allowed, const Tables* tb,
                                                      uint32_t qerr_lane, uint32_t pair_base, uint32_t ec_lo,
                                                      uint32_t ec_hi, uint32_t (&cw)[4], int (&didh)[2],
                                                      uint32_t (&Ech)[2]) {
  // ---- magnitudes, group maxima (4 elements = 2 registers), block maximum
  uint32_t a[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) a[i] = w[i] & 0x7fff7fffu;
  // per half of the lane's 32 elements (block size 32: both halves belong to one block):
  // biased exponent, the two bin scales of the Qvalue lookup, the chosen dialect's table address
  float sHh[2], sLh[2], magich[2];
  uint32_t finite = 1u;     // block size 32 without exponent clamp: 0 switches the value lookups off
  if (!B16) {
    uint32_t g2[4];   // (group 2q+1 max << 16) | group 2q max
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint32_t m0 = __vmaxu2(a[4 * q], a[4 * q + 1]);
      const uint32_t m1 = __vmaxu2(a[4 * q + 2], a[4 * q + 3]);
      g2[q] = __vmaxu2(__byte_perm(m0, m1, 0x5410), __byte_perm(m0, m1, 0x7632));
    }
    const uint32_t mm = __vmaxu2(__vmaxu2(g2[0], g2[1]), __vmaxu2(g2[2], g2[3]));
    uint32_t amax16 = max(mm & 0xffffu, mm >> 16);
    // An infinity or NaN in the block (inputs are required to be finite) must not turn into a table address out of
    // range.  The group maxima and the block maximum saturate at the largest finite bf16, so the exponent and the
    // error lookups stay in range; the value lookups further down are switched off for such a block (`finite` = 0).
    // Its output means nothing, but nothing is read or written out of bounds.  No branch: one in the middle of the
    // block's dependency chain cost the one-unit-per-lane kernels 3 to 15 %.
    // BRANCHY: the same protection as a rare branch that saturates every magnitude; cheaper (3 instead of 13
    // instructions per block) where a lane works on two blocks at a time and the branch does not hold anything up.
    if (!CLAMP && BRANCHY) {
      if (amax16 >= 0x7f80u) {
        amax16 = 0x7f7fu;
#pragma unroll
        for (int i = 0; i < 16; ++i) a[i] = __vminu2(a[i], 0x7f7f7f7fu);
#pragma unroll
        for (int q = 0; q < 4; ++q) g2[q] = __vminu2(g2[q], 0x7f7f7f7fu);
      }
    } else if (!CLAMP) {
      finite = amax16 < 0x7f80u ? 1u : 0u;
      amax16 = min(amax16, 0x7f7fu);
#pragma unroll
      for (int q = 0; q < 4; ++q) g2[q] = __vminu2(g2[q], 0x7f7f7f7fu);
      if (SEL == 1) {     // every element is a group maximum here
#pragma unroll
        for (int i = 0; i < 16; ++i) a[i] = __vminu2(a[i], 0x7f7f7f7fu);
      }
    }
    // ---- exponent: e = max(field,3) - 127 >= -124; element scale byte = field - 3
    uint32_t Ec = max(amax16 >> 7, 3u);
    if (CLAMP) {
      // clamped exponent range: magnitudes that would normalise to 16 or more saturate at the
      // largest value of bin 31 (biased exponent Ec, mantissa all ones)
      Ec = min(max(amax16 >> 7, ec_lo), ec_hi);
      const uint32_t bound = ((Ec << 7) | 0x7fu) * 0x10001u;
      amax16 = min(amax16, bound & 0xffffu);
#pragma unroll
      for (int i = 0; i < 16; ++i) a[i] = __vminu2(a[i], bound);
#pragma unroll
      for (int q = 0; q < 4; ++q) g2[q] = __vminu2(g2[q], bound);
    }
    const float s2 = __uint_as_float((257u - Ec) << 23);   // 2^(3-e)
    const float sG = s2 * 0x1p-21f;                        // bin in the mantissa of 2.0 + x
    const uint32_t bmax = __float_as_uint(__fmaf_rz(__uint_as_float(amax16 << 16), sG, 2.0f)) & 31u;
    // ---- dialect selection; the upper bf16 of a pair keeps the lower one as extra mantissa bits,
    // which truncation discards
    float gm[8];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      gm[2 * q] = bf16_lo_as_f32(g2[q]);
      gm[2 * q + 1] = __uint_as_float(g2[q]);
    }
    const int did = SEL == 1 ? choose_dialect_per_element<SEDA>(a, sG, bmax, allowed, tb, qerr_lane)
                    : SEL == 2 ? choose_dialect_all<SEDA>(gm, sG, allowed, tb, qerr_lane)
                               : choose_dialect<SEDA>(gm, sG, bmax, allowed, tb, qerr_lane);
    Ech[0] = Ech[1] = Ec;
    sHh[0] = sHh[1] = s2 * 0x1p-25f;                       // bin in the mantissa of 0.125 + x
    sLh[0] = sLh[1] = s2 * 0x1p-5f;                        // bin in the mantissa of 2^17 + x
    didh[0] = didh[1] = did;
  } else {
    // block size 16: the lane's two halves are two blocks; a group is the two elements of one register
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      uint32_t gx[8];   // group maximum in both halves of the register
#pragma unroll
      for (int k = 0; k < 8; ++k) gx[k] = __vmaxu2(a[8 * h + k], __byte_perm(a[8 * h + k], 0u, 0x1032));
      uint32_t mm = __vmaxu2(__vmaxu2(__vmaxu2(gx[0], gx[1]), __vmaxu2(gx[2], gx[3])),
                             __vmaxu2(__vmaxu2(gx[4], gx[5]), __vmaxu2(gx[6], gx[7])));
      if (!CLAMP && (mm & 0xffffu) >= 0x7f80u) {      // an infinity or NaN: saturate, as for block size 32
        mm = 0x7f7f7f7fu;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          a[8 * h + k] = __vminu2(a[8 * h + k], 0x7f7f7f7fu);
          gx[k] = __vminu2(gx[k], 0x7f7f7f7fu);
        }
      }
      uint32_t Ec = max((mm & 0xffffu) >> 7, 3u);
      if (CLAMP) {
        Ec = min(max((mm & 0xffffu) >> 7, ec_lo), ec_hi);
        const uint32_t bound = ((Ec << 7) | 0x7fu) * 0x10001u;
        mm = __vminu2(mm, bound);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          a[8 * h + k] = __vminu2(a[8 * h + k], bound);
          gx[k] = __vminu2(gx[k], bound);
        }
      }
      const float s2 = __uint_as_float((257u - Ec) << 23);
      const float sG = s2 * 0x1p-21f;
      const uint32_t bmax = __float_as_uint(__fmaf_rz(__uint_as_float(mm), sG, 2.0f)) & 31u;
      float gm[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) gm[k] = __uint_as_float(gx[k]);   // the low copy is truncated away
      Ech[h] = Ec;
      sHh[h] = s2 * 0x1p-25f;
      sLh[h] = s2 * 0x1p-5f;
      didh[h] = SEL == 2 ? choose_dialect_all<SEDA>(gm, sG, allowed, tb, qerr_lane)
                         : choose_dialect<SEDA>(gm, sG, bmax, allowed, tb, qerr_lane);
    }
  }
  // ---- Qvalue: one lookup per element pair.  124*36 + 144 = 9*512, so the exponent fields of
  // 36*bits(0.125 + ..) + bits(2^17 + ..) cancel mod 2^32 and leave table + 36*bin_hi + bin_lo.
  magich[0] = __uint_as_float(0x48000000u + pair_base + (uint32_t)didh[0] * kPairStride);
  magich[1] = B16 ? __uint_as_float(0x48000000u + pair_base + (uint32_t)didh[1] * kPairStride) : magich[0];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int h = B16 ? (q >> 1) : 0;
    uint32_t b[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t av = a[4 * q + j];
      const uint32_t th = __float_as_uint(__fmaf_rz(__uint_as_float(av), sHh[h], 0.125f));
      const uint32_t tl = __float_as_uint(__fmaf_rz(bf16_lo_as_f32(av), sLh[h], magich[h]));
      if (B16 || CLAMP || BRANCHY) {
        b[j] = lds_u8(th * (uint32_t)kPairMul + tl);
      } else {
        b[j] = th;      // any defined value: the load replaces it unless the block holds an infinity or NaN
        lds_u8_if(b[j], th * (uint32_t)kPairMul + tl, finite);
      }
    }
    const uint32_t idx = b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24);
    // sign bits: byte masks by sign replication, then to bit 3 of every nibble
    const uint32_t sa = prmt(w[4 * q], w[4 * q + 1], 0xfdb9u);
    const uint32_t sb = prmt(w[4 * q + 2], w[4 * q + 3], 0xfdb9u);
    const uint32_t ev = __byte_perm(sa, sb, 0x6420), od = __byte_perm(sa, sb, 0x7531);
    cw[q] = idx | (((ev & 0x0f0f0f0fu) | (od & 0xf0f0f0f0u)) & 0x88888888u);
  }
}

// What a lane needs besides the tables: its column of the error table and the base of the pair table.
struct Lane {
  uint32_t qerr_lane;
  uint32_t pair_base;
};
__device__ __forceinline__ Lane lane_state(const Tables* tb) {
  Lane ln;
  ln.qerr_lane = smem_u32(tb->qerr_private) + ((uint32_t)threadIdx.x & 15u) * 8u;
  ln.pair_base = smem_u32(tb->pairlut);
  return ln;
}

// Copies the table image into shared memory with all threads of the CTA (16-byte accesses); the caller
// synchronises the CTA before the first use.
__device__ __forceinline__ void copy_tables(Tables* dst, const void* image) {
  const uint4* src = static_cast<const uint4*>(image);
  uint4* d = reinterpret_cast<uint4*>(dst);
  const int n = (int)(sizeof(Tables) / 16);
  const int nthreads = blockDim.x * blockDim.y * blockDim.z;
  const int tid = threadIdx.x + blockDim.x * (threadIdx.y + blockDim.y * threadIdx.z);
  for (int i = tid; i < n; i += nthreads) d[i] = src[i];
}

// One block of 32 fp32 values in registers -> 4 code words and the metadata record.  Every value is taken
// as it is (nothing is rounded to bf16): only its upper 16 bits enter, which fix sign, scale exponent
// and the 0.5-wide bin of the value.  allowed = SeDA mask of the token (all ones: unconstrained).
template <bool SEDA = false>
__device__ __forceinline__ void quantize_block_f32(const float (&x)[32], uint32_t allowed, const Tables* tb, const Lane& ln,
                                                   uint32_t (&codes)[4], uint16_t* meta) {
  uint32_t w[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) w[i] = __byte_perm(__float_as_uint(x[2 * i]), __float_as_uint(x[2 * i + 1]), 0x7632);
  int did[2];
  uint32_t Eb[2];
  quantize_packed_block<SEDA, false, false>(w, allowed ? allowed : 1u, tb, ln.qerr_lane, ln.pair_base, 3u, 254u, codes, did, Eb);
  *meta = (uint16_t)((Eb[0] - 3u) | ((uint32_t)did[0] << 8));
}

}  // namespace fb4blk

#endif  // FB4_BLOCK_CUH_
