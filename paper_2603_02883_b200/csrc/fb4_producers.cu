// Producers fused in front of the FB4 quantizer (App. D.2: the quantizer runs as the tail of the preceding
// operation): the per-channel affine step and LayerNorm + modulation, on the TMA-staged ring and the block
// routine of the quantize kernels.  The producer's result y exists only in registers.
#include <cuda.h>

#include "fb4_block.cuh"
#include "fb4_device.cuh"
#include "fb4_internal.h"
#include "fb4_staging.cuh"

namespace {

using namespace fb4blk;
using namespace fb4stage;

// ---------------------------------------------------------------------------------------------
// Per-channel affine producer fused in front of the quantizer (App. D.2: quantization fused with the
// preceding operation; the elementwise tail of a LayerNorm, or the modulation of an adaLN block):
// y = x * g_c + bias_c in fp32 (one FMA, g_c = gain_c or 1 + gain_c), quantized from registers with
// quantize_packed_block (on the upper 16 bits of y); y never reaches HBM.  Same ring, tables and tile shape as the bf16 kernel, but
// the warps are column-stationary: a warp keeps one tile column (1024 channels) and walks down the
// rows, so each lane holds the gain and bias of its 32 channels in 32 registers (two bf16 per
// register) for the whole launch.  Warps beyond a multiple of the number of tile columns stay idle.
// SEDA: the token's cluster mask restricts the candidates (Sec. 3.4); it is fetched one tile ahead.
// MX: the result leaves as e4m3 bytes + E8M0 scales (p.e4m3 / p.scales) instead of codes / metadata.
template <bool PLUS_ONE, bool SEDA, bool MX = false>
__global__ void __launch_bounds__(kWarps * 32, 1)
fb4_quantize_affine_kernel(const __grid_constant__ CUtensorMap tmap, const SmemTables* __restrict__ g_tables,
                           FastParams p, const uint16_t* __restrict__ gain, const uint16_t* __restrict__ bias,
                           int64_t n_active, Fb4RowExtras ex) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* ring = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  SmemTables* tb = reinterpret_cast<SmemTables*>(ring + kWarps * kStages * kTileBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(tb) + sizeof(SmemTables));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t gwarp = (int64_t)blockIdx.x * kWarps + warp;
  const int32_t tpr = (int32_t)p.tiles_per_row;

  const uint32_t table_bar = smem_u32(bars + kWarps * kStages);
  // every warp initialises its own ring barriers; the first thread also the table barrier, and it
  // starts the table copy at once (one thread doing all kWarps * kStages + 1 inits in a row used to
  // hold the whole CTA for most of a microsecond)
  if (lane == 0) {
    for (int i = 0; i < kStages; ++i) mbar_init(smem_u32(bars + warp * kStages + i), 1);
    if (warp == 0) mbar_init(table_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (warp == 0) {
      mbar_expect_tx(table_bar, (uint32_t)sizeof(SmemTables));
      bulk_load(smem_u32(tb), g_tables, (uint32_t)sizeof(SmemTables), table_bar);
    }
  }
  __syncthreads();

  const uint32_t my_ring = smem_u32(ring + (size_t)warp * kStages * kTileBytes);
  const uint32_t my_bars = smem_u32(bars + warp * kStages);
  // this warp's tiles: column `col`, rows row0, row0 + rstep, ...
  const int32_t rstep = (int32_t)(n_active / tpr);
  const int32_t col = (int32_t)(gwarp % tpr);
  const int64_t row0 = gwarp / tpr;
  const int32_t n_mine = (gwarp < n_active && row0 < p.T) ? (int32_t)((p.T - row0 + rstep - 1) / rstep) : 0;
  int64_t pre_row = row0;
  int32_t it_pre = 0;
#pragma unroll
  for (int s = 0; s < kStages; ++s) {
    if (it_pre < n_mine && lane == 0) {
      mbar_expect_tx(my_bars + 8 * s, kTileBytes);
      tma_load_tile(my_ring + s * kTileBytes, &tmap, my_bars + 8 * s, col * 16, (int)pre_row);
    }
    ++it_pre;
    pre_row += rstep;
  }
  const int64_t nblk = p.C >> 5;
  const int64_t blk = (int64_t)col * 32 + lane;
  const bool active = blk < nblk;
  // gain and bias of this lane's 32 channels: fac[i] = gain bits | bias bits << 16
  uint32_t fac[32];
  {
    uint32_t gw[16], bw[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) gw[k] = bw[k] = 0u;
    if (active && n_mine > 0) {
      const uint4* gp = reinterpret_cast<const uint4*>(gain + blk * 32);
      const uint4* bp = reinterpret_cast<const uint4*>(bias + blk * 32);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint4 g = __ldg(gp + q), b = __ldg(bp + q);
        gw[4 * q] = g.x; gw[4 * q + 1] = g.y; gw[4 * q + 2] = g.z; gw[4 * q + 3] = g.w;
        bw[4 * q] = b.x; bw[4 * q + 1] = b.y; bw[4 * q + 2] = b.z; bw[4 * q + 3] = b.w;
      }
    }
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      fac[2 * k] = (gw[k] & 0xffffu) | (bw[k] << 16);
      fac[2 * k + 1] = (gw[k] >> 16) | (bw[k] & 0xffff0000u);
    }
  }
  {
    uint32_t spins = 0;
    bool ready = mbar_try_wait(table_bar, 0u);
    while (!ready && ++spins < kSpinLimit) ready = mbar_try_wait(table_bar, 0u);
    if (!__all_sync(0xffffffffu, ready)) {
      if (lane == 0) atomicOr(p.status, 1u);
      for (int j = 0; j < kStages && j < n_mine; ++j) {
        uint32_t tries = 0;
        while (!mbar_try_wait(my_bars + 8 * j, 0u) && ++tries < kSpinLimit) {}
      }
      return;
    }
  }
  const uint32_t pair_base = smem_u32(tb->pairlut);
  const uint32_t qerr_base = smem_u32(tb->qerr_private) + ((uint32_t)lane & 15u) * 8u;
  const uint32_t r = (uint32_t)lane >> 1, c0 = ((uint32_t)lane & 1u) * 4u;
  uint32_t chunk_off[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) chunk_off[j] = r * 128u + (((c0 + j) ^ (r & 7u)) << 4);
  const int64_t code_row_bytes = p.C >> 1;

  // cluster mask of a row; an id outside [-1, n_clusters) counts as -1 and is reported
  bool bad_cid = false;
  auto row_mask = [&](int64_t t) -> uint32_t {
    const int32_t cid = __ldg(ex.cluster_id + t);
    if ((uint32_t)cid < (uint32_t)ex.n_clusters) {
      const uint32_t m = __ldg(ex.cluster_mask + cid);
      return m ? m : 1u;   // a zero mask (precondition violated) yields dialect 0
    }
    if (cid != -1) bad_cid = true;
    return 0xffffffffu;
  };
  uint32_t mask_next = 0xffffffffu;
  if (SEDA && n_mine > 0) mask_next = row_mask(row0);

  int s = 0;
  uint32_t parity = 0;
  int64_t row = row0;
  for (int32_t it = 0; it < n_mine; ++it) {
    const uint32_t allowed = mask_next;
    if (SEDA && it + 1 < n_mine) mask_next = row_mask(row + rstep);
    const uint32_t bar = my_bars + 8 * s;
    uint32_t spins = 0;
    bool ready = mbar_try_wait(bar, parity);
    while (!ready && ++spins < kSpinLimit) ready = mbar_try_wait(bar, parity);
    if (!__all_sync(0xffffffffu, ready)) {
      if (lane == 0) atomicOr(p.status, 1u);
      int sj = s;
      uint32_t pj = parity;
      for (int j = 1; j < kStages; ++j) {
        if (it + j >= n_mine) break;
        if (++sj == kStages) { sj = 0; pj ^= 1u; }
        uint32_t tries = 0;
        while (!mbar_try_wait(my_bars + 8 * sj, pj) && ++tries < kSpinLimit) {}
      }
      break;
    }
    uint32_t yw[16];   // y cut to its upper 16 bits, two per register
    {
      const uint32_t base = my_ring + s * kTileBytes;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint4 v = lds_v4(base + chunk_off[q]);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint32_t y[2];
#pragma unroll
          for (int hlf = 0; hlf < 2; ++hlf) {
            // x as float32 by the mixed-precision add (x + -0 = x): the FMA pipe instead of a shift or mask on
            // the busier ALU pipe
            const float xv = hlf ? bf16_plus_f32<1>(w[j], -0.0f) : bf16_plus_f32<0>(w[j], -0.0f);
            const uint32_t f = fac[8 * q + 2 * j + hlf];
            float g = __uint_as_float(f << 16);
            if (PLUS_ONE) g = __fadd_rn(1.0f, g);
            y[hlf] = __float_as_uint(__fmaf_rn(xv, g, __uint_as_float(f & 0xffff0000u)));
          }
          yw[4 * q + j] = __byte_perm(y[0], y[1], 0x7632);
        }
      }
    }
    uint32_t cw[4], Eb[2];
    int did[2];
    quantize_packed_block<SEDA, false, false>(yw, allowed, tb, qerr_base, pair_base, 3u, 254u, cw, did, Eb);
    const uint32_t m = (Eb[0] - 3u) | ((uint32_t)did[0] << 8);
    if (MX) {
      if (active) {
        const uint2 fb = tb->fb_e4m3[did[0]];
        uint32_t o[8];
#pragma unroll
        for (int q = 0; q < 4; ++q) fb4dev::codes_to_e4m3(cw[q], fb, o[2 * q], o[2 * q + 1]);
        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p.e4m3 + row * p.C + blk * 32),
                     "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
        p.scales[fb4dev::mx_scale_offset(row, blk, nblk, p.scale_col_tiles, p.scale_tiled)] = (uint8_t)m;
      }
    } else if (active) {
      *reinterpret_cast<uint4*>(p.codes + row * code_row_bytes + blk * 16) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
      p.meta[row * nblk + blk] = (uint16_t)m;
    }
    __syncwarp();
    if (lane == 0 && it_pre < n_mine) {
      mbar_expect_tx(bar, kTileBytes);
      tma_load_tile(my_ring + s * kTileBytes, &tmap, bar, col * 16, (int)pre_row);
    }
    ++it_pre;
    pre_row += rstep;
    row += rstep;
    if (++s == kStages) { s = 0; parity ^= 1u; }
  }
  if (SEDA && bad_cid && lane == 0) atomicOr(p.status, 2u);
}

// ---------------------------------------------------------------------------------------------
// The same producer on the flat tiles, for contiguous tensors whose tokens are whole tiles (C a multiple of
// 1024): the flat kernel's loop with one unit per lane (2 KB tiles, four stages, stage addresses as immediates,
// output addresses linear in the unit number) and a grid whose warp count is a multiple of the tiles per token,
// so a warp still keeps its tile column - and its lanes the factors of their 32 channels - while it walks down
// the tokens.
template <bool PLUS_ONE, bool SEDA, bool MX = false>
__global__ void __launch_bounds__(kWarps * 32, 1)
fb4_quantize_affine_flat_kernel(const __grid_constant__ CUtensorMap tmap, const SmemTables* __restrict__ g_tables,
                                FlatParams p, const uint16_t* __restrict__ gain, const uint16_t* __restrict__ bias,
                                Fb4RowExtras ex) {
  constexpr int kSt = kStages;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* ring = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  SmemTables* tb = reinterpret_cast<SmemTables*>(ring + kWarps * kStages * kTileBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(tb) + sizeof(SmemTables));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t g0 = blockIdx.x * kWarps + warp;
  const uint32_t wstride = gridDim.x * kWarps;          // a multiple of the tiles per token (chosen by the host)
  const uint32_t tpr = p.units_row >> 5;                // tiles per token
  const uint32_t table_bar = smem_u32(bars + kWarps * kStages);
  if (lane == 0) {
    for (int i = 0; i < kSt; ++i) mbar_init(smem_u32(bars + warp * kStages + i), 1);
    if (warp == 0) mbar_init(table_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (warp == 0) {
      mbar_expect_tx(table_bar, (uint32_t)sizeof(SmemTables));
      bulk_load(smem_u32(tb), g_tables, (uint32_t)sizeof(SmemTables), table_bar);
    }
  }
  __syncthreads();
  const uint32_t my_ring = smem_u32(ring + (size_t)warp * kStages * kTileBytes);
  const uint32_t my_bars = smem_u32(bars + warp * kStages);
  const int32_t n_mine = g0 < p.n_tiles ? (int32_t)((p.n_tiles - g0 + wstride - 1) / wstride) : 0;
  int32_t y_pre = (int32_t)(g0 * 16u);                  // first 128-byte row of the next tile to request
  const int32_t y_step = (int32_t)(wstride * 16u);
#pragma unroll
  for (int s = 0; s < kSt; ++s) {
    if (s < n_mine && lane == 0) {
      mbar_expect_tx(my_bars + 8 * s, kTileBytes);
      tma_load_2d(my_ring + s * kTileBytes, &tmap, my_bars + 8 * s, 0, y_pre);
    }
    y_pre += y_step;
  }
  const uint32_t col = g0 % tpr;                        // this warp's tile column, for the whole launch
  uint32_t row = g0 / tpr;
  const uint32_t row_step = wstride / tpr;
  const uint32_t rem = col * 32u + (uint32_t)lane;      // this lane's unit inside a token = its block of channels
  uint32_t unit = g0 * 32u + (uint32_t)lane;
  const uint32_t unit_step = wstride * 32u;
  // gain and bias of this lane's 32 channels: fac[i] = gain bits | bias bits << 16
  uint32_t fac[32];
  {
    uint32_t gw[16], bw[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) gw[k] = bw[k] = 0u;
    if (n_mine > 0) {
      const uint4* gp = reinterpret_cast<const uint4*>(gain + (size_t)rem * 32);
      const uint4* bp = reinterpret_cast<const uint4*>(bias + (size_t)rem * 32);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint4 g = __ldg(gp + q), b = __ldg(bp + q);
        gw[4 * q] = g.x; gw[4 * q + 1] = g.y; gw[4 * q + 2] = g.z; gw[4 * q + 3] = g.w;
        bw[4 * q] = b.x; bw[4 * q + 1] = b.y; bw[4 * q + 2] = b.z; bw[4 * q + 3] = b.w;
      }
    }
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      fac[2 * k] = (gw[k] & 0xffffu) | (bw[k] << 16);
      fac[2 * k + 1] = (gw[k] >> 16) | (bw[k] & 0xffff0000u);
    }
  }
  {
    uint32_t spins = 0;
    bool ready = mbar_try_wait(table_bar, 0u);
    while (!ready && ++spins < kSpinLimit) ready = mbar_try_wait(table_bar, 0u);
    if (!__all_sync(0xffffffffu, ready)) {
      if (lane == 0) atomicOr(p.status, 1u);
      for (int j = 0; j < kSt && j < n_mine; ++j) {
        uint32_t tries = 0;
        while (!mbar_try_wait(my_bars + 8 * j, 0u) && ++tries < kSpinLimit) {}
      }
      return;
    }
  }
  const uint32_t pair_base = smem_u32(tb->pairlut);
  const uint32_t qerr_base = smem_u32(tb->qerr_private) + ((uint32_t)lane & 15u) * 8u;
  uint32_t chunk[4];      // this lane's 16-byte chunks in stage 0: row lane / 2, chunks (lane & 1) * 4 + j
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint32_t r = (uint32_t)lane >> 1, c = ((uint32_t)lane & 1u) * 4u + (uint32_t)j;
    chunk[j] = my_ring + r * 128u + ((c ^ (r & 7u)) << 4);
  }
  // cluster mask of a token, fetched one tile ahead; an id outside [-1, n_clusters) counts as -1 and is reported
  bool bad_cid = false;
  auto row_mask = [&](uint32_t t) -> uint32_t {
    const int32_t cid = __ldg(ex.cluster_id + t);
    if ((uint32_t)cid < (uint32_t)ex.n_clusters) {
      const uint32_t m = __ldg(ex.cluster_mask + cid);
      return m ? m : 1u;   // a zero mask (precondition violated) yields dialect 0
    }
    if (cid != -1) bad_cid = true;
    return 0xffffffffu;
  };
  uint32_t mask_next = 0xffffffffu;
  if (SEDA && n_mine > 0) mask_next = row_mask(row);

  uint32_t parity = 0;
  bool failed = false;
  for (int32_t it = 0; it < n_mine && !failed; it += kSt) {
#pragma unroll
    for (int s = 0; s < kSt; ++s) {
      if (it + s < n_mine && !failed) {
        const uint32_t allowed = mask_next;
        if (SEDA && it + s + 1 < n_mine) mask_next = row_mask(row + row_step);
        const uint32_t bar = my_bars + 8 * s;
        uint32_t spins = 0;
        bool ready = mbar_try_wait(bar, parity);
        while (!ready && ++spins < kSpinLimit) ready = mbar_try_wait(bar, parity);
        if (!__all_sync(0xffffffffu, ready)) {
          // A load never arrived: raise the status bit, give the loads still in flight for this warp a
          // bounded chance to land, stop.
          if (lane == 0) atomicOr(p.status, 1u);
          for (int j = 1; j < kSt; ++j) {
            if (it + s + j >= n_mine) break;
            const int sj = (s + j) % kSt;
            const uint32_t pj = (s + j) >= kSt ? (parity ^ 1u) : parity;
            uint32_t tries = 0;
            while (!mbar_try_wait(my_bars + 8 * sj, pj) && ++tries < kSpinLimit) {}
          }
          failed = true;
        } else {
          uint32_t yw[16];     // y cut to its upper 16 bits, two per register
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint4 v = lds_v4(chunk[q] + s * kTileBytes);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              uint32_t y[2];
#pragma unroll
              for (int hlf = 0; hlf < 2; ++hlf) {
                const float xv = hlf ? bf16_plus_f32<1>(w[j], -0.0f) : bf16_plus_f32<0>(w[j], -0.0f);
                const uint32_t f = fac[8 * q + 2 * j + hlf];
                float g = __uint_as_float(f << 16);
                if (PLUS_ONE) g = __fadd_rn(1.0f, g);
                y[hlf] = __float_as_uint(__fmaf_rn(xv, g, __uint_as_float(f & 0xffff0000u)));
              }
              yw[4 * q + j] = __byte_perm(y[0], y[1], 0x7632);
            }
          }
          uint32_t cw[4], Eb[2];
          int did[2];
          quantize_packed_block<SEDA, false, false>(yw, allowed, tb, qerr_base, pair_base, 3u, 254u, cw, did, Eb);
          const uint32_t m = (Eb[0] - 3u) | ((uint32_t)did[0] << 8);
          if (unit < p.n_units) {
            if (MX) {
              const uint2 fb = tb->fb_e4m3[did[0]];
              uint32_t o[8];
#pragma unroll
              for (int q = 0; q < 4; ++q) fb4dev::codes_to_e4m3(cw[q], fb, o[2 * q], o[2 * q + 1]);
              stg_v8(p.e4m3 + (size_t)unit * 32u, o);
              const int64_t so = p.scale_tiled ? fb4dev::mx_scale_offset(row, rem, p.units_row, p.scale_col_tiles, 1)
                                               : (int64_t)unit;
              p.scales[so] = (uint8_t)m;
            } else {
              *reinterpret_cast<uint4*>(p.codes + (size_t)unit * 16u) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
              p.meta[unit] = (uint16_t)m;
            }
          }
          // ---- refill this stage (all lanes have consumed their registers from it)
          __syncwarp();
          if (lane == 0 && it + s + kSt < n_mine) {
            mbar_expect_tx(bar, kTileBytes);
            tma_load_2d(my_ring + s * kTileBytes, &tmap, bar, 0, y_pre);
          }
          y_pre += y_step;
          unit += unit_step;
          row += row_step;
        }
      }
    }
    parity ^= 1u;
  }
  if (SEDA && bad_cid && lane == 0) atomicOr(p.status, 2u);
}

// ---------------------------------------------------------------------------------------------
// LayerNorm + per-channel modulation fused in front of the quantizer (App. D.2 names LayerNorm as an
// operation the quantizer runs behind; the adaLN blocks modulate the normalised activation as
// y = n * (1 + scale_c) + shift_c).  A token's C channels (a multiple of 1024, at most 16 384) belong to
// C / 1024 warps of one CTA, lane = one block of 32 channels, held in registers (as the 16 packed input
// words) from the load to the code store: the row is read once, y never exists in memory.  Every float32
// operation is rounded once and the additions have a fixed order, so the result is reproducible bit for bit:
//   block sums in channel order; the 32 block sums of a warp by an xor butterfly (offsets 16 .. 1; all
//   lanes end with the same bits because a + b = b + a); the warp sums of a token added to +0 in warp order;
//   mean = total / C; d = x - mean; sums of squares with q = fma(d, d, q), same reduction; var = total / C;
//   rstd = 1 / sqrt(var + eps) (correctly rounded root and division); y = fma(d * rstd, g, b).
// Same ring and tables as the flat kernel with one unit per lane; gain and bias of a lane's channels stay
// in registers for the whole launch (a lane keeps its block column).  The warp sums travel through shared
// memory behind two CTA barriers per step, and between barriers every chain of additions is a latency
// chain, so a step takes TWO tokens per team of warps (a CTA takes 2 * 16 / (C / 1024) tokens per step):
// the chains of the two tokens interleave and a token costs one barrier.
struct LnParams {
  uint32_t T;
  uint32_t units_row;      // C / 32
  uint32_t wpr;            // warps per token = C / 1024
  uint32_t teams;          // teams of wpr warps per CTA; a team takes two tokens per step
  float c_f32;             // (float)C
  float eps;
  uint8_t* codes;
  uint16_t* meta;
  uint32_t* status;
};

// NW = warps per CTA: 12 where the warps of a token divide 12 (170 registers per thread, room for two tokens and
// the factors), 16 otherwise.
template <bool PLUS_ONE, bool SEDA, int NW>
__global__ void __launch_bounds__(NW * 32, 1)
fb4_quantize_layernorm_kernel(const __grid_constant__ CUtensorMap tmap, const SmemTables* __restrict__ g_tables,
                              LnParams p, const uint16_t* __restrict__ gain, const uint16_t* __restrict__ bias,
                              Fb4RowExtras ex) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* ring = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  SmemTables* tb = reinterpret_cast<SmemTables*>(ring + kWarps * kStages * kTileBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(tb) + sizeof(SmemTables));
  // warp sums: [2 passes][2 tokens][team][16], a team's entries padded with +0 to 16 (written once, below)
  float* part = reinterpret_cast<float*>(bars + kWarps * kStages + 2);      // 16-byte aligned: the barriers are an odd count
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t team = (uint32_t)warp / p.wpr, wcol = (uint32_t)warp % p.wpr;
  const bool warp_used = team < p.teams;

  const uint32_t table_bar = smem_u32(bars + kWarps * kStages);
  if (lane == 0) {
    for (int i = 0; i < kStages; ++i) mbar_init(smem_u32(bars + warp * kStages + i), 1);
    if (warp == 0) mbar_init(table_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (warp == 0) {
      mbar_expect_tx(table_bar, (uint32_t)sizeof(SmemTables));
      bulk_load(smem_u32(tb), g_tables, (uint32_t)sizeof(SmemTables), table_bar);
    }
  }
  for (int i = threadIdx.x; i < 4 * kWarps * 16; i += blockDim.x) part[i] = 0.0f;
  __syncthreads();
  const uint32_t my_ring = smem_u32(ring + (size_t)warp * kStages * kTileBytes);
  const uint32_t my_bars = smem_u32(bars + warp * kStages);
  // Step i of this CTA covers the token pairs (blockIdx.x + i * gridDim.x) * teams + team; a pair is the tokens
  // 2 * pair and 2 * pair + 1.  Ring stage 2 * (i mod 2) + ab holds this warp's 1024 channels of token ab of step i.
  const uint32_t n_pairs = (p.T + 1u) / 2u;
  const uint32_t n_sets = (n_pairs + p.teams - 1) / p.teams;
  const int32_t n_steps = blockIdx.x < n_sets ? (int32_t)((n_sets - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0;
  const uint32_t pair0 = blockIdx.x * p.teams + team;
  const uint32_t pair_step = gridDim.x * p.teams;
  auto row_of = [&](int32_t i, int ab) -> uint64_t { return 2u * ((uint64_t)pair0 + (uint64_t)i * pair_step) + (uint64_t)ab; };
  auto tile_valid = [&](int32_t i, int ab) -> bool { return warp_used && i < n_steps && row_of(i, ab) < p.T; };
  const uint32_t rows128 = p.units_row / 2;      // 128-byte rows of the 2-D view per token
  auto request = [&](int32_t i, int ab) {
    const uint32_t st = (uint32_t)(2 * (i & 1) + ab);
    mbar_expect_tx(my_bars + 8 * st, kTileBytes);
    tma_load_2d(my_ring + st * kTileBytes, &tmap, my_bars + 8 * st, 0, (int)((uint32_t)row_of(i, ab) * rows128 + wcol * 16u));
  };
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int ab = 0; ab < 2; ++ab)
        if (tile_valid(i, ab)) request(i, ab);
  }
  // this lane's 32 channels: the factor g = gain or 1 + gain in float32, the bias as loaded (two bf16 per register)
  float gf[32];
  uint32_t bw[16];
  {
    uint32_t gw[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) gw[k] = bw[k] = 0u;
    if (warp_used) {
      const uint4* gp = reinterpret_cast<const uint4*>(gain + ((size_t)wcol * 32 + lane) * 32);
      const uint4* bp = reinterpret_cast<const uint4*>(bias + ((size_t)wcol * 32 + lane) * 32);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint4 g = __ldg(gp + q), b = __ldg(bp + q);
        gw[4 * q] = g.x; gw[4 * q + 1] = g.y; gw[4 * q + 2] = g.z; gw[4 * q + 3] = g.w;
        bw[4 * q] = b.x; bw[4 * q + 1] = b.y; bw[4 * q + 2] = b.z; bw[4 * q + 3] = b.w;
      }
    }
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      gf[2 * k] = __uint_as_float(gw[k] << 16);
      gf[2 * k + 1] = __uint_as_float(gw[k] & 0xffff0000u);
      if (PLUS_ONE) {
        gf[2 * k] = __fadd_rn(1.0f, gf[2 * k]);
        gf[2 * k + 1] = __fadd_rn(1.0f, gf[2 * k + 1]);
      }
    }
  }
  bool tables_ok;
  {
    uint32_t spins = 0;
    bool ready = mbar_try_wait(table_bar, 0u);
    while (!ready && ++spins < kSpinLimit) ready = mbar_try_wait(table_bar, 0u);
    tables_ok = __all_sync(0xffffffffu, ready);
  }
  const uint32_t pair_base = smem_u32(tb->pairlut);
  const uint32_t qerr_base = smem_u32(tb->qerr_private) + ((uint32_t)lane & 15u) * 8u;
  const uint32_t r = (uint32_t)lane >> 1, c0 = ((uint32_t)lane & 1u) * 4u;
  uint32_t chunk_off[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) chunk_off[j] = r * 128u + (((c0 + j) ^ (r & 7u)) << 4);
  // the warp sums of this warp's team, added to +0 in warp order; the entries behind the team's last warp hold +0,
  // which leaves the sum as it is, so whole groups of four are read and added
  auto team_total = [&](const float* ps) -> float {
    const float4* v4 = reinterpret_cast<const float4*>(ps + team * 16u);
    float t = 0.0f;
#pragma unroll
    for (int k4 = 0; k4 < kWarps / 4; ++k4) {
      if ((uint32_t)(4 * k4) >= p.wpr) break;
      const float4 v = v4[k4];
      t = __fadd_rn(__fadd_rn(__fadd_rn(__fadd_rn(t, v.x), v.y), v.z), v.w);
    }
    return t;
  };
  // The warps of a team meet at a barrier of their own (hardware barrier 1 + team), so the teams of a CTA drift
  // apart and one team's additions overlap another team's quantization; warps outside every team meet nobody.
  auto team_sync = [&]() {
    if (warp_used) asm volatile("bar.sync %0, %1;" ::"r"(team + 1u), "r"(p.wpr * 32u) : "memory");
  };
  bool bad_cid = false;
  // A wait that ran out (tables or a tile) is remembered per warp; the warp keeps meeting its team's barriers
  // but neither reads nor writes data any more, and the status bit is raised.
  bool dead = !tables_ok;
  uint32_t parity = 0, parity_dead = 0;
  int32_t it_dead = 0;
  for (int32_t it = 0; it < n_steps; ++it) {
    if (!dead) { parity_dead = parity; it_dead = it; }   // where the ring stood when the warp gave up
    const uint32_t st0 = (uint32_t)(2 * (it & 1));
    bool live[2];
    uint32_t allowed[2] = {0xffffffffu, 0xffffffffu};
    uint32_t w[2][16];       // the two tokens' blocks as loaded: two bf16 per register
#pragma unroll
    for (int ab = 0; ab < 2; ++ab) {
      live[ab] = tile_valid(it, ab) && !dead;
#pragma unroll
      for (int k = 0; k < 16; ++k) w[ab][k] = 0u;
      if (SEDA && live[ab]) {
        const int32_t cid = __ldg(ex.cluster_id + row_of(it, ab));
        if ((uint32_t)cid < (uint32_t)ex.n_clusters) {
          const uint32_t m = __ldg(ex.cluster_mask + cid);
          allowed[ab] = m ? m : 1u;
        } else if (cid != -1) {
          bad_cid = true;
        }
      }
    }
#pragma unroll
    for (int ab = 0; ab < 2; ++ab) {
      if (live[ab]) {      // warp-uniform
        const uint32_t bar = my_bars + 8 * (st0 + ab);
        uint32_t spins = 0;
        bool ready = mbar_try_wait(bar, parity);
        while (!ready && ++spins < kSpinLimit) ready = mbar_try_wait(bar, parity);
        if (!__all_sync(0xffffffffu, ready)) {
          dead = true;
          live[0] = live[1] = false;
        } else {
          const uint32_t base = my_ring + (st0 + ab) * kTileBytes;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint4 v = lds_v4(base + chunk_off[q]);
            w[ab][4 * q] = v.x; w[ab][4 * q + 1] = v.y; w[ab][4 * q + 2] = v.z; w[ab][4 * q + 3] = v.w;
          }
        }
      }
    }
    // ---- mean: block sum in channel order, butterfly over the warp, warp sums of the token in order
    float sum[2];
#pragma unroll
    for (int ab = 0; ab < 2; ++ab) {
      float s = __uint_as_float(w[ab][0] << 16);
      s = bf16_plus_f32<1>(w[ab][0], s);
#pragma unroll
      for (int k = 1; k < 16; ++k) {
        s = bf16_plus_f32<0>(w[ab][k], s);
        s = bf16_plus_f32<1>(w[ab][k], s);
      }
      sum[ab] = s;
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
#pragma unroll
      for (int ab = 0; ab < 2; ++ab) sum[ab] = __fadd_rn(sum[ab], __shfl_xor_sync(0xffffffffu, sum[ab], off));
    }
    if (lane == 0 && warp_used) {
      part[team * 16u + wcol] = sum[0];
      part[kWarps * 16 + team * 16u + wcol] = sum[1];
    }
    team_sync();
    float mean[2] = {0.0f, 0.0f};
    if (warp_used) {
#pragma unroll
      for (int ab = 0; ab < 2; ++ab) mean[ab] = __fdiv_rn(team_total(part + ab * kWarps * 16), p.c_f32);
    }
    // ---- variance
    float q[2] = {0.0f, 0.0f};
#pragma unroll
    for (int k = 0; k < 16; ++k) {
#pragma unroll
      for (int ab = 0; ab < 2; ++ab) {
        const float d0 = bf16_minus_f32<0>(w[ab][k], mean[ab]);
        q[ab] = __fmaf_rn(d0, d0, q[ab]);
        const float d1 = bf16_minus_f32<1>(w[ab][k], mean[ab]);
        q[ab] = __fmaf_rn(d1, d1, q[ab]);
      }
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
#pragma unroll
      for (int ab = 0; ab < 2; ++ab) q[ab] = __fadd_rn(q[ab], __shfl_xor_sync(0xffffffffu, q[ab], off));
    }
    if (lane == 0 && warp_used) {
      part[2 * kWarps * 16 + team * 16u + wcol] = q[0];
      part[3 * kWarps * 16 + team * 16u + wcol] = q[1];
    }
    team_sync();
#pragma unroll
    for (int ab = 0; ab < 2; ++ab) {
      if (live[ab]) {
        const float var = __fdiv_rn(team_total(part + (2 + ab) * kWarps * 16), p.c_f32);
        const float rstd = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(var, p.eps)));
        // ---- modulation, cut to the upper 16 bits (all the quantizer needs), quantize, store
        uint32_t yw[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          uint32_t y[2];
#pragma unroll
          for (int hlf = 0; hlf < 2; ++hlf) {
            const float dv = hlf ? bf16_minus_f32<1>(w[ab][k], mean[ab]) : bf16_minus_f32<0>(w[ab][k], mean[ab]);
            const float bv = __uint_as_float(hlf ? (bw[k] & 0xffff0000u) : (bw[k] << 16));
            y[hlf] = __float_as_uint(__fmaf_rn(__fmul_rn(dv, rstd), gf[2 * k + hlf], bv));
          }
          yw[k] = __byte_perm(y[0], y[1], 0x7632);
        }
        uint32_t cw[4], Eb[2];
        int did[2];
        quantize_packed_block<SEDA, false, false>(yw, allowed[ab], tb, qerr_base, pair_base, 3u, 254u, cw, did, Eb);
        const size_t unit = (size_t)row_of(it, ab) * p.units_row + wcol * 32u + (uint32_t)lane;
        *reinterpret_cast<uint4*>(p.codes + unit * 16u) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
        p.meta[unit] = (uint16_t)((Eb[0] - 3u) | ((uint32_t)did[0] << 8));
      }
    }
    // ---- refill the two stages of this step with the tokens two steps ahead
    __syncwarp();
    if (lane == 0 && !dead) {
#pragma unroll
      for (int ab = 0; ab < 2; ++ab)
        if (tile_valid(it + 2, ab)) request(it + 2, ab);
    }
    if (it & 1) parity ^= 1u;
  }
  if (dead) {
    if (lane == 0) atomicOr(p.status, 1u);
    // the loads still in flight for this warp (the tokens of the step it gave up at and of the next one) get a
    // bounded chance to land before the CTA's shared memory goes
    for (int j = 0; j < 2; ++j) {
      const uint32_t pj = ((it_dead & 1) + j) >= 2 ? (parity_dead ^ 1u) : parity_dead;
      for (int ab = 0; ab < 2; ++ab) {
        if (!tile_valid(it_dead + j, ab)) continue;
        const uint32_t st = (uint32_t)(2 * ((it_dead + j) & 1) + ab);
        uint32_t tries = 0;
        while (!mbar_try_wait(my_bars + 8 * st, pj) && ++tries < kSpinLimit) {}
      }
    }
  }
  if (SEDA && bad_cid && lane == 0) atomicOr(p.status, 2u);
}

constexpr size_t kSmemBytesLn =
    1024 + (size_t)kWarps * kStages * kTileBytes + sizeof(SmemTables) + (kWarps * kStages + 2) * 8 + 4 * kWarps * 16 * sizeof(float);
static_assert(kSmemBytesLn <= 227 * 1024, "shared memory budget of one CTA");

}  // namespace

// Opt in to the kernels' dynamic shared memory on the current device (once per context).
cudaError_t fb4_producers_prepare_device() {
  const int bytes = (int)kSmemBytes;
  const cudaFuncAttribute attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
  cudaError_t e = cudaSuccess;
#define FB4_OPT_IN(...) \
  if (e == cudaSuccess) e = cudaFuncSetAttribute(fb4_quantize_affine_kernel<__VA_ARGS__>, attr, bytes); \
  if (e == cudaSuccess) e = cudaFuncSetAttribute(fb4_quantize_affine_flat_kernel<__VA_ARGS__>, attr, bytes)
  FB4_OPT_IN(false, false, false); FB4_OPT_IN(true, false, false); FB4_OPT_IN(false, true, false); FB4_OPT_IN(true, true, false);
  FB4_OPT_IN(false, false, true); FB4_OPT_IN(true, false, true); FB4_OPT_IN(false, true, true); FB4_OPT_IN(true, true, true);
#undef FB4_OPT_IN
#define FB4_OPT_IN(...) \
  if (e == cudaSuccess) e = cudaFuncSetAttribute(fb4_quantize_layernorm_kernel<__VA_ARGS__>, attr, (int)kSmemBytesLn)
  FB4_OPT_IN(false, false, 12); FB4_OPT_IN(true, false, 12); FB4_OPT_IN(false, true, 12); FB4_OPT_IN(true, true, 12);
  FB4_OPT_IN(false, false, 16); FB4_OPT_IN(true, false, 16); FB4_OPT_IN(false, true, 16); FB4_OPT_IN(true, true, 16);
#undef FB4_OPT_IN
  return e;
}

// Affine producer + quantizer in one pass: default configuration only, and at most as many tile
// columns as the grid has warps (every warp keeps one tile column).
bool fb4_fast_affine_eligible(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, const void* gain,
                              const void* bias) {
  if (!fb4_fast_mx_eligible(ctx, x, T, C, ld)) return false;
  if ((reinterpret_cast<uintptr_t>(gain) & 15) || (reinterpret_cast<uintptr_t>(bias) & 15)) return false;
  return (C + 1023) / 1024 <= (int64_t)ctx->sm_count * kWarps;
}

cudaError_t fb4_launch_quantize_fast_affine(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld,
                                            const void* gain, const void* bias, int plus_one,
                                            const Fb4RowExtras& ex, uint8_t* codes, uint16_t* meta,
                                            cudaStream_t stream, uint8_t* e4m3, uint8_t* scales, int tiled) {
  const SmemTables* tables = static_cast<const SmemTables*>(ctx->d_fast_tables);
  const uint16_t* g = static_cast<const uint16_t*>(gain);
  const uint16_t* b = static_cast<const uint16_t*>(bias);
  CUtensorMap map;
  // Contiguous tensors whose tokens are whole tiles take the flat tiles, on the largest grid whose warps are a
  // multiple of the tiles per token (147 CTAs for 12 or 3 tiles per token on 148 SMs).
  if (fb4_flat_eligible(T, C, ld) && C % 1024 == 0) {
    const int64_t tpr = C / 1024, n_tiles = T * tpr;
    int64_t fgrid = (n_tiles + kWarps - 1) / kWarps;
    if (fgrid > ctx->sm_count) fgrid = ctx->sm_count;
    while (fgrid > 0 && (fgrid * kWarps) % tpr != 0) --fgrid;
    if (fgrid > 0 && fgrid * 8 >= ctx->sm_count * 7) {     // else too few SMs would work: the strided kernel below
      FlatParams fp;
      int unused = 0;
      const cudaError_t fe = fb4_flat_setup(ctx, x, T, C, true, false, &map, &fp, &unused);   // one unit per lane
      if (fe != cudaSuccess) return fe;
      fp.codes = codes;
      fp.meta = meta;
      if (e4m3) {   // MXFP8 output: padding of the tiled scale layout = scale 1, the kernel writes real entries only
        fp.e4m3 = e4m3;
        fp.scales = scales;
        fp.scale_tiled = tiled;
        const int64_t n_col = C / 32;
        fp.scale_col_tiles = (n_col + 3) / 4;
        if (tiled && ((T & 127) || (n_col & 3))) {
          const cudaError_t me =
              cudaMemsetAsync(scales, 0x7f, (size_t)(((T + 127) / 128) * fp.scale_col_tiles * 512), stream);
          if (me != cudaSuccess) return me;
        }
      }
#define FB4_AFFINE_FLAT(P, S, M)                                                                                   \
  fb4_quantize_affine_flat_kernel<P, S, M><<<(int)fgrid, kWarps * 32, kSmemBytes, stream>>>(map, tables, fp, g, b, ex)
      switch ((plus_one ? 1 : 0) | (ex.cluster_id ? 2 : 0) | (e4m3 ? 4 : 0)) {
        case 0: FB4_AFFINE_FLAT(false, false, false); break;
        case 1: FB4_AFFINE_FLAT(true, false, false); break;
        case 2: FB4_AFFINE_FLAT(false, true, false); break;
        case 3: FB4_AFFINE_FLAT(true, true, false); break;
        case 4: FB4_AFFINE_FLAT(false, false, true); break;
        case 5: FB4_AFFINE_FLAT(true, false, true); break;
        case 6: FB4_AFFINE_FLAT(false, true, true); break;
        default: FB4_AFFINE_FLAT(true, true, true); break;
      }
#undef FB4_AFFINE_FLAT
      return cudaGetLastError();
    }
  }
  FastParams p;
  int grid = 0;
  const cudaError_t e = fb4_fast_setup(ctx, x, T, C, ld, false, &map, &p, &grid);
  if (e != cudaSuccess) return e;
  p.codes = codes;
  p.meta = meta;
  // column-stationary warps: the largest multiple of the tile columns that the grid's warps cover;
  // enough CTAs for one warp per (row, tile column) and never fewer than one full set of columns
  const int64_t tpr = p.tiles_per_row;
  int64_t want = (p.n_tiles + kWarps - 1) / kWarps;
  const int64_t min_ctas = (tpr + kWarps - 1) / kWarps;
  if (want < min_ctas) want = min_ctas;
  grid = (int)(want < ctx->sm_count ? want : ctx->sm_count);
  const int64_t n_active = ((int64_t)grid * kWarps / tpr) * tpr;
  if (n_active <= 0) return cudaErrorInvalidValue;
  if (e4m3) {   // MXFP8 output: padding of the tiled scale layout = scale 1, the kernel writes real entries only
    p.e4m3 = e4m3;
    p.scales = scales;
    p.scale_tiled = tiled;
    const int64_t n_col = C / 32;
    p.scale_col_tiles = (n_col + 3) / 4;
    if (tiled && ((T & 127) || (n_col & 3))) {
      const cudaError_t me =
          cudaMemsetAsync(scales, 0x7f, (size_t)(((T + 127) / 128) * p.scale_col_tiles * 512), stream);
      if (me != cudaSuccess) return me;
    }
  }
#define FB4_AFFINE(P, S, M) \
  fb4_quantize_affine_kernel<P, S, M><<<grid, kWarps * 32, kSmemBytes, stream>>>(map, tables, p, g, b, n_active, ex)
  switch ((plus_one ? 1 : 0) | (ex.cluster_id ? 2 : 0) | (e4m3 ? 4 : 0)) {
    case 0: FB4_AFFINE(false, false, false); break;
    case 1: FB4_AFFINE(true, false, false); break;
    case 2: FB4_AFFINE(false, true, false); break;
    case 3: FB4_AFFINE(true, true, false); break;
    case 4: FB4_AFFINE(false, false, true); break;
    case 5: FB4_AFFINE(true, false, true); break;
    case 6: FB4_AFFINE(false, true, true); break;
    default: FB4_AFFINE(true, true, true); break;
  }
#undef FB4_AFFINE
  return cudaGetLastError();
}


// LayerNorm producer + quantizer in one pass: default configuration, contiguous rows, C a multiple of 1024
// and at most 16 384 (one warp per 1024 channels, a token inside one CTA).
bool fb4_fast_layernorm_eligible(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, const void* gain,
                                 const void* bias) {
  if (!fb4_fast_mx_eligible(ctx, x, T, C, ld)) return false;
  if ((reinterpret_cast<uintptr_t>(gain) & 15) || (reinterpret_cast<uintptr_t>(bias) & 15)) return false;
  return fb4_flat_eligible(T, C, ld) && C % 1024 == 0 && C <= 1024 * kWarps;
}

cudaError_t fb4_launch_quantize_layernorm(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, const void* gain,
                                          const void* bias, int plus_one, float eps, const Fb4RowExtras& ex,
                                          uint8_t* codes, uint16_t* meta, cudaStream_t stream) {
  CUtensorMap map;
  FlatParams fp;
  int grid = 0;
  const cudaError_t e = fb4_flat_setup(ctx, x, T, C, true, false, &map, &fp, &grid);   // one unit per lane: 2 KB tiles
  if (e != cudaSuccess) return e;
  LnParams p{};
  p.T = (uint32_t)T;
  p.units_row = (uint32_t)(C / 32);
  p.wpr = (uint32_t)(C / 1024);
  const int nw = (12 % p.wpr == 0) ? 12 : kWarps;
  p.teams = (uint32_t)nw / p.wpr;
  p.c_f32 = (float)C;
  p.eps = eps;
  p.codes = codes;
  p.meta = meta;
  p.status = ctx->d_status;
  const int64_t n_sets = ((T + 1) / 2 + p.teams - 1) / p.teams;      // a team takes two tokens per step
  grid = (int)(n_sets < ctx->sm_count ? n_sets : ctx->sm_count);
  const SmemTables* tables = static_cast<const SmemTables*>(ctx->d_fast_tables);
  const uint16_t* g = static_cast<const uint16_t*>(gain);
  const uint16_t* b = static_cast<const uint16_t*>(bias);
#define FB4_LN(P, S) \
  do { \
    if (nw == 12) fb4_quantize_layernorm_kernel<P, S, 12><<<grid, 12 * 32, kSmemBytesLn, stream>>>(map, tables, p, g, b, ex); \
    else fb4_quantize_layernorm_kernel<P, S, 16><<<grid, 16 * 32, kSmemBytesLn, stream>>>(map, tables, p, g, b, ex); \
  } while (0)
  switch ((plus_one ? 1 : 0) | (ex.cluster_id ? 2 : 0)) {
    case 0: FB4_LN(false, false); break;
    case 1: FB4_LN(true, false); break;
    case 2: FB4_LN(false, true); break;
    default: FB4_LN(true, true); break;
  }
#undef FB4_LN
  return cudaGetLastError();
}
