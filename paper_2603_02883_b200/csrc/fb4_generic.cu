// Generic FB4 quantize kernel: one thread per block, any supported configuration
// (block size 16/32, num_groups 8 or = block size, clamped exponent ranges, both
// selection modes, arbitrary SeDA masks, residual pass for salient tokens).
// It is the path for shapes/configurations the TMA-staged kernel does not take.
//
// Per block (Sec. 3.1-3.2): amax -> exponent e -> v = |x| * 2^(3-e) -> bin = floor(2v)
// -> group maxima (as bins; the bin map is monotone) -> stage-1 candidate mask
// -> sum of Qerror over the group maxima for every candidate -> argmin
// -> Qvalue lookup per element -> packed 4-bit codes + (dialect id, scale byte).
#include "fb4_internal.h"

namespace {

struct SmemTables {
  uint8_t qvalue[32][32];
  uint8_t qerror[32][32];
  uint8_t fb[32][8];
  uint32_t stage1[32];
};
static_assert(sizeof(SmemTables) == sizeof(Fb4DeviceTables), "table layouts must match");

struct GenericParams {
  int exp_min, exp_max, select_all;
};

// 2^k for k in [-149, 127]
__device__ __forceinline__ float pow2f(int k) {
  return k >= -126 ? __int_as_float((k + 127) << 23) : __int_as_float(1 << (k + 149));
}

// One block: ax = magnitudes, sgn bit i = sign of element i.  Writes packed nibbles.
template <int B, int GS>
__device__ __forceinline__ void quantize_block(const float (&ax)[B], uint32_t sgn, const SmemTables& tb,
                                               const GenericParams& p, uint32_t allowed, uint32_t (&packed)[B / 8],
                                               int& did, int& e_out) {
  constexpr int G = B / GS;
  float amax = 0.f;
#pragma unroll
  for (int i = 0; i < B; ++i) amax = fmaxf(amax, ax[i]);
  // floor(log2(amax)) is the exponent field; zero and subnormal maxima clamp to exp_min (>= -124)
  int e = amax == 0.f ? p.exp_min : (int)((__float_as_uint(amax) >> 23) & 0xff) - 127;
  e = max(p.exp_min, min(p.exp_max, e));
  // bin = floor(2 * |x| * 2^(3-e)), saturated at 31.  Magnitudes that would normalise to 16 or more
  // (possible only when the exponent was clamped from above) are first cut to the largest fp32 below
  // 2^(e+1); then 2v < 32 and the bin is read from the low mantissa bits of 2.0 + 2v * 2^-22, formed
  // by one round-toward-zero FMA (exact: no conversion instruction, no intermediate rounding).
  const float cut = __uint_as_float(((uint32_t)(e + 128) << 23) - 1u);
  const float sG = pow2f(3 - e) * 0x1p-21f;   // 3-e-21 in [-145,106]
  uint8_t bin[B];
#pragma unroll
  for (int i = 0; i < B; ++i)
    bin[i] = (uint8_t)(__float_as_uint(__fmaf_rz(fminf(ax[i], cut), sG, 2.0f)) & 31u);
  uint8_t gb[G];
  int bmax = 0;
#pragma unroll
  for (int g = 0; g < G; ++g) {
    int m = 0;
#pragma unroll
    for (int i = 0; i < GS; ++i) m = max(m, (int)bin[g * GS + i]);
    gb[g] = (uint8_t)m;
    bmax = max(bmax, m);
  }
  uint32_t cand = allowed;
  if (!p.select_all) {
    cand = tb.stage1[bmax] & allowed;
    if (cand == 0) cand = allowed;
  }
  int best = 0, best_err = 0x7fffffff;
  for (uint32_t m = cand; m; m &= m - 1) {
    const int d = __ffs((int)m) - 1;
    int err = 0;
#pragma unroll
    for (int g = 0; g < G; ++g) err += tb.qerror[d][gb[g]];
    if (err < best_err) { best_err = err; best = d; }   // ascending d: ties keep the lowest id
  }
#pragma unroll
  for (int w = 0; w < B / 8; ++w) {
    uint32_t word = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int k = w * 8 + i;
      const uint32_t nib = tb.qvalue[best][bin[k]] | (((sgn >> k) & 1u) << 3);
      word |= nib << (4 * i);
    }
    packed[w] = word;
  }
  did = best;
  e_out = e;
}

template <int B>
__device__ __forceinline__ void store_block(const uint32_t (&packed)[B / 8], int did, int e, uint8_t* codes_row,
                                            uint16_t* meta_row, int64_t blk) {
  if constexpr (B == 32) {
    *reinterpret_cast<uint4*>(codes_row + blk * 16) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
  } else {
    *reinterpret_cast<uint2*>(codes_row + blk * 8) = make_uint2(packed[0], packed[1]);
  }
  meta_row[blk] = (uint16_t)((e + 124) | (did << 8));
}

// row index of token t in the compact salient list, or -1
__device__ __forceinline__ int64_t salient_row(const Fb4RowExtras& ex, int64_t t) {
  if (ex.n_salient <= 0) return -1;
  if (ex.tile > 0) {
    const int64_t s = t / ex.tile;
    return (s < ex.n_salient && ex.salient_idx[s] == (int32_t)t) ? s : -1;
  }
  int64_t lo = 0, hi = ex.n_salient - 1;
  while (lo <= hi) {
    const int64_t mid = (lo + hi) >> 1;
    const int32_t v = ex.salient_idx[mid];
    if (v == (int32_t)t) return mid;
    if (v < (int32_t)t) lo = mid + 1; else hi = mid - 1;
  }
  return -1;
}

// MOD 1 / 2: bf16 input goes through the per-channel affine producer first, y = x * g_c + bias_c in
// fp32 with g_c = gain_c (1) or 1 + gain_c (2), one FMA; the block is quantized from y (App. D.2).
template <int B, int GS, bool F32, bool RESID, int MOD = 0>
__global__ void __launch_bounds__(128)
fb4_quantize_generic_kernel(const void* __restrict__ xin, int64_t T, int64_t C, int64_t ld,
                            const Fb4DeviceTables* __restrict__ tables, GenericParams p, Fb4RowExtras ex,
                            uint8_t* __restrict__ codes, uint16_t* __restrict__ meta, uint32_t* __restrict__ status,
                            const uint16_t* __restrict__ gain = nullptr, const uint16_t* __restrict__ bias = nullptr) {
  __shared__ SmemTables tb;
  {
    const uint32_t* src = reinterpret_cast<const uint32_t*>(tables);
    uint32_t* dst = reinterpret_cast<uint32_t*>(&tb);
    for (int i = threadIdx.x; i < (int)(sizeof(SmemTables) / 4); i += blockDim.x) dst[i] = src[i];
  }
  __syncthreads();
  const int64_t nblk = C / B;
  const int64_t total = T * nblk;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t id = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; id < total; id += stride) {
    const int64_t t = id / nblk;
    const int64_t blk = id - t * nblk;
    float xs[B], ax[B];
    uint32_t sgn = 0;
    if (F32) {   // fp32 input: the values as they are
      const uint4* src = reinterpret_cast<const uint4*>(static_cast<const float*>(xin) + t * ld + blk * B);
#pragma unroll
      for (int q = 0; q < B / 4; ++q) {
        const uint4 v = src[q];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          xs[q * 4 + j] = __uint_as_float(w[j]);
          sgn |= (w[j] >> 31) << (q * 4 + j);
        }
      }
    }
    const uint4* src = reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(xin) + t * ld + blk * B);
#pragma unroll
    for (int q = 0; q < (F32 ? 0 : B / 8); ++q) {
      const uint4 v = src[q];
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t lo = w[j] << 16, hi = w[j] & 0xffff0000u;
        xs[q * 8 + 2 * j] = __uint_as_float(lo);
        xs[q * 8 + 2 * j + 1] = __uint_as_float(hi);
        sgn |= (lo >> 31) << (q * 8 + 2 * j);
        sgn |= (hi >> 31) << (q * 8 + 2 * j + 1);
      }
    }
    if (MOD != 0) {
      sgn = 0;
#pragma unroll
      for (int i = 0; i < B; ++i) {
        const int64_t c = blk * B + i;
        float g = __uint_as_float((uint32_t)gain[c] << 16);
        if (MOD == 2) g = __fadd_rn(1.0f, g);
        xs[i] = __fmaf_rn(xs[i], g, __uint_as_float((uint32_t)bias[c] << 16));
        sgn |= (__float_as_uint(xs[i]) >> 31) << i;
      }
    }
#pragma unroll
    for (int i = 0; i < B; ++i) ax[i] = fabsf(xs[i]);
    uint32_t allowed = 0xffffffffu;
    if (ex.cluster_id) {
      const int32_t cid = ex.cluster_id[t];
      if ((uint32_t)cid < (uint32_t)ex.n_clusters) allowed = ex.cluster_mask[cid];
      else if (cid != -1) atomicOr(status, 2u);   // out of range: unconstrained, reported in the status word
      if (allowed == 0) allowed = 1u;   // precondition violated: stay in bounds
    }
    uint32_t packed[B / 8];
    int did, e;
    quantize_block<B, GS>(ax, sgn, tb, p, allowed, packed, did, e);
    store_block<B>(packed, did, e, codes + t * (C / 2), meta + t * nblk, blk);

    const int64_t srow = RESID ? salient_row(ex, t) : -1;
    if (RESID && srow >= 0) {
      // Sec. 3.3: Delta = x - Q(x), exact in fp32 for the default exponent range; quantized again
      const float sc = pow2f(e - 3);
      uint32_t dsgn = 0;
#pragma unroll
      for (int i = 0; i < B; ++i) {
        const uint32_t nib = (packed[i / 8] >> (4 * (i % 8))) & 15u;
        const float mag = (float)tb.fb[did][nib & 7u] * sc;
        const float delta = __fsub_rn(xs[i], (nib & 8u) ? -mag : mag);
        dsgn |= (__float_as_uint(delta) >> 31) << i;
        ax[i] = fabsf(delta);
      }
      uint32_t rpacked[B / 8];
      int rdid, re;
      quantize_block<B, GS>(ax, dsgn, tb, p, allowed, rpacked, rdid, re);
      store_block<B>(rpacked, rdid, re, ex.res_codes + srow * (C / 2), ex.res_meta + srow * nblk, blk);
    }
  }
}

}  // namespace

cudaError_t fb4_launch_quantize_generic(const fb4_ctx* ctx, const void* x, int x_is_f32, int64_t T, int64_t C,
                                        int64_t ld, const Fb4RowExtras& ex, uint8_t* codes, uint16_t* meta,
                                        cudaStream_t stream, const void* gain, const void* bias, int plus_one) {
  const int B = (int)ctx->cfg.block_size, G = (int)ctx->cfg.num_groups;
  const int64_t total = T * (C / B);
  if (total == 0) return cudaSuccess;
  GenericParams p{ctx->cfg.exp_min, ctx->cfg.exp_max, ctx->cfg.select_mode == 1 ? 1 : 0};
  const int threads = 128;
  int64_t want = (total + threads - 1) / threads;
  const int64_t cap = 0x7fffffff;   // one block of work per thread, CTAs dispatched in order (see fb4_decode.cu)
  const int grid = (int)(want < cap ? want : cap);
  const bool resid = ex.n_salient > 0;
#define FB4_LAUNCH_K(BB, GSZ, F, R) \
  fb4_quantize_generic_kernel<BB, GSZ, F, R><<<grid, threads, 0, stream>>>(x, T, C, ld, ctx->d_tables, p, ex, codes, meta, \
                                                                           ctx->d_status)
  const uint16_t* g16 = static_cast<const uint16_t*>(gain);
  const uint16_t* b16 = static_cast<const uint16_t*>(bias);
  if (gain && (x_is_f32 || resid)) return cudaErrorInvalidValue;
#define FB4_LAUNCH_MOD(BB, GSZ, M)                                                                       \
  fb4_quantize_generic_kernel<BB, GSZ, false, false, M><<<grid, threads, 0, stream>>>(x, T, C, ld, ctx->d_tables, p, ex, \
                                                                                      codes, meta, ctx->d_status, g16, b16)
#define FB4_LAUNCH(BB, GSZ)                                  \
  do {                                                       \
    if (gain && plus_one) FB4_LAUNCH_MOD(BB, GSZ, 2);        \
    else if (gain) FB4_LAUNCH_MOD(BB, GSZ, 1);               \
    else if (x_is_f32) FB4_LAUNCH_K(BB, GSZ, true, false);   \
    else if (resid) FB4_LAUNCH_K(BB, GSZ, false, true);      \
    else FB4_LAUNCH_K(BB, GSZ, false, false);                \
  } while (0)
  if (B == 32 && G == 8) FB4_LAUNCH(32, 4);
  else if (B == 32 && G == 32) FB4_LAUNCH(32, 1);
  else if (B == 16 && G == 8) FB4_LAUNCH(16, 2);
  else if (B == 16 && G == 16) FB4_LAUNCH(16, 1);
  else return cudaErrorInvalidValue;
#undef FB4_LAUNCH
#undef FB4_LAUNCH_MOD
#undef FB4_LAUNCH_K
  return cudaGetLastError();
}
