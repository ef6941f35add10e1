// TMA-staged FB4 quantize kernels for sm_100a: num_groups 8, two-stage selection, block size 32
// or 16, any exponent clamp, with the SeDA restriction and the residual pass of salient tokens
// fused in (template parameters), plus a variant for fp32 input.
//
// Work unit: a tile of 1024 consecutive channels of one token (2 KB of bf16 = 32 blocks).
// Every warp owns a ring of shared-memory stages; lane 0 keeps the ring full with 3-D TMA
// loads (tensor view [T][C/64][64], box 1 x 16 x 64, 128-byte swizzle) that complete on
// per-stage mbarriers.  Lane i then quantizes block i of the tile entirely in registers:
// it reads its 64 bytes with four conflict-free 16-byte shared loads, and the warp writes
// 512 B of codes and 64 B of metadata with one coalesced store each.  With block size 16 a
// lane's 64 bytes are two blocks.  The lookup tables (75 KB, built on the host at init) arrive by
// one bulk asynchronous copy per CTA.  Every wait on an mbarrier is bounded and raises a status
// bit when it runs out.
//
// Arithmetic (all exact):
//  * magnitudes are compared as 15-bit integers (bf16 patterns are monotone), two per register;
//  * bin = floor(2 * |x| * 2^(3-e)) is read from the low mantissa bits of a round-toward-zero
//    FMA against a power-of-two constant; for the upper bf16 of a register pair the lower
//    half may stay in place as extra mantissa bits because truncation discards it;
//  * Qerror: one 64-bit word per (stage-1 group, bin) holds the error of up to 8 candidate
//    dialects as bytes, so 8 loads + packed adds score all candidates; argmin on (err<<3|j);
//  * Qvalue: a per-dialect table indexed by the bins of TWO elements returns a finished code
//    byte; its address comes out of one integer multiply-add of the two FMA results, whose
//    exponent bits are chosen to cancel modulo 2^32.
#include <cuda.h>

#include <cstring>
#include <mutex>
#include <new>

#include "fb4_block.cuh"
#include "fb4_device.cuh"
#include "fb4_internal.h"
#include "fb4_staging.cuh"

namespace {

using fb4dev::pow2f;
using fb4dev::prmt;
using namespace fb4blk;
using namespace fb4stage;

// Residual pass of the lane's block(s) (Sec. 3.3): Delta = x - Q(x) in fp32 (exact for the full
// exponent range, the correctly rounded difference otherwise), quantized again with the same tables
// as the main pass, from the upper 16 bits of every Delta (see quantize_packed_block).
// w = the 16 input registers (2 bf16 each), cw = the 4 code words, didh / Ech = dialect and biased
// exponent per half (equal halves for block size 32).
template <bool SEDA, bool B16, bool CLAMP, int SEL = 0, bool BRANCHY = false>
__device__ __forceinline__ void residual_block(const uint32_t* w, const uint32_t* cw, const int* didh,
                                               const uint32_t* Ech, uint32_t allowed, const SmemTables* tb,
                                               uint32_t qerr_lane, uint32_t pair_base, uint32_t ec_lo, uint32_t ec_hi,
                                               uint32_t* rcw, uint32_t* rmeta) {
  uint32_t dw[16];     // Delta cut to its upper 16 bits, two per register like the input
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int h = B16 ? (q >> 1) : 0;
    const uint4 dt = tb->fb_bf16[didh[h]];
    const uint32_t sc2 = fb4dev::scale_bf16x2(Ech[h] - 3u);   // element scale 2^(e-3) as two bf16
    uint32_t xh[4];    // Q(x) of the word's 8 elements, two bf16 per register, signs included
    fb4dev::decode_word(cw[q], dt, sc2, xh);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t xw = w[4 * q + j];
      // x - Q(x) by the mixed-precision add and sub (the halves are read where they lie; same bits as the
      // float32 subtraction of the unpacked values)
      const uint32_t d0 = __float_as_uint(bf16_minus_f32<0>(xw, bf16_plus_f32<0>(xh[j], -0.0f)));
      const uint32_t d1 = __float_as_uint(bf16_minus_f32<1>(xw, bf16_plus_f32<1>(xh[j], -0.0f)));
      dw[4 * q + j] = __byte_perm(d0, d1, 0x7632);
    }
  }
  uint32_t rc[4], rE[2];
  int rd[2];
  quantize_packed_block<SEDA, B16, CLAMP, SEL, BRANCHY>(dw, allowed, tb, qerr_lane, pair_base, ec_lo, ec_hi, rc, rd, rE);
#pragma unroll
  for (int q = 0; q < 4; ++q) rcw[q] = rc[q];
  *rmeta = B16 ? (((rE[0] - 3u) | ((uint32_t)rd[0] << 8)) | (((rE[1] - 3u) | ((uint32_t)rd[1] << 8)) << 16))
               : ((rE[0] - 3u) | ((uint32_t)rd[0] << 8));
}

struct TilePos {
  int32_t row;         // T < 2^31
  int32_t col;
  __device__ __forceinline__ void advance(const FastParams& p, int32_t tiles_per_row) {
    row += (int32_t)p.step_rows;
    col += p.step_cols;
    if (col >= tiles_per_row) { col -= tiles_per_row; ++row; }
  }
};

template <bool SEDA, bool DECOMP, bool B16, bool CLAMP, bool MX = false>
__global__ void __launch_bounds__(kWarps * 32, 1)
fb4_quantize_fast_kernel(const __grid_constant__ CUtensorMap tmap, const SmemTables* __restrict__ g_tables,
                         FastParams p, Fb4RowExtras ex) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // [ring: kWarps*kStages*2048 B, 1 KB aligned for the 128-byte swizzle][tables][mbarriers: one per
  // stage of every warp, then one for the tables]
  uint8_t* ring = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  SmemTables* tb = reinterpret_cast<SmemTables*>(ring + kWarps * kStages * kTileBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(tb) + sizeof(SmemTables));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Tile -> warp assignment.  Plain and SeDA calls: tile g goes to warp g mod (all warps of the grid),
  // so the whole grid sweeps the tensor as one front.  Calls with a residual pass: every CTA takes a
  // contiguous range of tiles and deals it round-robin to its own warps, which spreads the (much
  // more expensive) tiles of a salient token over many warps and gives every CTA the same share
  // of salient tokens.
  int64_t gwarp, g_end, wstride;
  if (DECOMP) {
    const int64_t per = p.n_tiles / gridDim.x, extra = p.n_tiles % gridDim.x, b = blockIdx.x;
    const int64_t t0 = b * per + (b < extra ? b : extra);
    gwarp = t0 + warp;
    g_end = t0 + per + (b < extra ? 1 : 0);
    wstride = kWarps;
  } else {
    gwarp = (int64_t)blockIdx.x * kWarps + warp;
    g_end = p.n_tiles;
    wstride = (int64_t)gridDim.x * kWarps;
  }
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
  TilePos cur, pre;   // tile being quantized; next tile to request
  cur.row = (int32_t)(gwarp / tpr);
  cur.col = (int32_t)(gwarp - (int64_t)cur.row * tpr);
  pre = cur;
  // this warp's tiles are gwarp, gwarp + wstride, ...: n_mine of them, counted in 32 bits
  const int32_t n_mine = gwarp < g_end ? (int32_t)((g_end - gwarp + wstride - 1) / wstride) : 0;
  int32_t it_pre = 0;   // iteration whose tile `pre` points at
  const bool use_seda = SEDA && ex.cluster_id != nullptr;
  // Per-token extras travel in register queues, fetched as far ahead as the tile data: entry k
  // belongs to the tile k steps ahead.  cidq = cluster id; the cluster mask follows its id two steps
  // behind.
  int32_t cidq[kStages];
  // prologue: fill the ring
#pragma unroll
  for (int s = 0; s < kStages; ++s) {
    cidq[s] = -1;
    if (it_pre < n_mine) {
      if (lane == 0) {
        mbar_expect_tx(my_bars + 8 * s, kTileBytes);
        tma_load_tile(my_ring + s * kTileBytes, &tmap, my_bars + 8 * s, pre.col * 16, pre.row);
      }
      if (use_seda) cidq[s] = ex.cluster_id[pre.row];
    }
    ++it_pre;
    pre.advance(p, tpr);
  }
  // salient tokens: an ascending list (one per tile, or given by the caller); this warp's rows never
  // decrease, so a cursor walks it.  Position of the first entry >= this warp's first row:
  int64_t list_pos = 0;
  int32_t list_next = 0x7fffffff;
  if (DECOMP && n_mine > 0) {
    int64_t lo = 0, hi = ex.n_salient;
    while (lo < hi) {
      const int64_t mid = (lo + hi) >> 1;
      if (ex.salient_idx[mid] < cur.row) lo = mid + 1; else hi = mid;
    }
    list_pos = lo;
    if (lo < ex.n_salient) list_next = ex.salient_idx[lo];
  }
  // a cluster id outside [-1, n_clusters) is treated as -1 (unconstrained) and reported in bit 1 of
  // the status word when the warp is done: the mask table is never read out of bounds
  const uint32_t n_cl = (uint32_t)ex.n_clusters;
  bool bad_cid = false;
  uint32_t maskq[2] = {0xffffffffu, 0xffffffffu};
  if (use_seda) {
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      if ((uint32_t)cidq[k] < n_cl) maskq[k] = ex.cluster_mask[cidq[k]];
      else if (cidq[k] != -1) bad_cid = true;
    }
  }
  // ---- the tables arrive behind the first tile loads; bounded wait like every other wait here
  {
    uint32_t spins = 0;
    bool ready = mbar_try_wait(table_bar, 0u);
    while (!ready && ++spins < kSpinLimit) ready = mbar_try_wait(table_bar, 0u);
    if (!__all_sync(0xffffffffu, ready)) {
      if (lane == 0) atomicOr(p.status, 1u);
      // give this warp's tile loads a bounded chance to land before the CTA's shared memory goes
      for (int j = 0; j < kStages && j < n_mine; ++j) {
        uint32_t tries = 0;
        while (!mbar_try_wait(my_bars + 8 * j, 0u) && ++tries < kSpinLimit) {}
      }
      return;
    }
  }

  const uint32_t pair_base = smem_u32(tb->pairlut);
  const uint32_t qerr_base = smem_u32(tb->qerr_private) + ((uint32_t)lane & 15u) * 8u;
  // this lane's 64 bytes inside a stage: row r = lane/2 of 128 B, chunks (lane&1)*4 + j, swizzled by r&7
  const uint32_t r = (uint32_t)lane >> 1, c0 = ((uint32_t)lane & 1u) * 4u;
  uint32_t chunk_off[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) chunk_off[j] = r * 128u + (((c0 + j) ^ (r & 7u)) << 4);

  const int64_t nblk = p.C >> 5;
  const int64_t code_row_bytes = p.C >> 1;

  int s = 0;
  uint32_t parity = 0;
  for (int32_t it = 0; it < n_mine; ++it) {
    // ---- fetch the extras of the tiles ahead (pre = the tile kStages steps ahead)
    int32_t cid_new = -1;
    uint32_t mask_new = 0xffffffffu;
    if (SEDA) {
      if (use_seda) {
        if (it_pre < n_mine) cid_new = ex.cluster_id[pre.row];
        if ((uint32_t)cidq[2] < n_cl) mask_new = ex.cluster_mask[cidq[2]];
        else if (cidq[2] != -1) bad_cid = true;
      }
    }

    const uint32_t bar = my_bars + 8 * s;
    uint32_t spins = 0;
    bool ready = mbar_try_wait(bar, parity);
    while (!ready && ++spins < kSpinLimit) ready = mbar_try_wait(bar, parity);
    if (!__all_sync(0xffffffffu, ready)) {
      // A load never arrived: raise the status bit, give the loads still in flight for this warp a
      // bounded chance to land (so none writes into shared memory after the CTA has gone), stop.
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
    const int64_t row = cur.row;   // 64-bit for the output offsets
    const int64_t blk = (int64_t)cur.col * 32 + lane;
    const bool active = blk < nblk;

    uint32_t w[16];
    {
      const uint32_t base = my_ring + s * kTileBytes;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint4 v = lds_v4(base + chunk_off[j]);
        w[4 * j] = v.x; w[4 * j + 1] = v.y; w[4 * j + 2] = v.z; w[4 * j + 3] = v.w;
      }
    }
    uint32_t cw[4], Ech[2];
    int didh[2];
    uint32_t allowed = 0xffffffffu;
    if (SEDA) {
      allowed = maskq[0];
      if (allowed == 0) allowed = 1u;   // precondition violated: stay in bounds
    }
    quantize_packed_block<SEDA, B16, CLAMP>(w, allowed, tb, qerr_base, pair_base, p.ec_lo, p.ec_hi, cw, didh, Ech);
    if (MX) {
      // MXFP8 output (block size 32): the codes become e4m3 bytes in registers, the scale byte is the
      // E8M0 scale; 32 contiguous bytes per lane, 1 KB per warp
      if (active) {
        const uint2 fb = tb->fb_e4m3[didh[0]];
        uint32_t o[8];
#pragma unroll
        for (int q = 0; q < 4; ++q) fb4dev::codes_to_e4m3(cw[q], fb, o[2 * q], o[2 * q + 1]);
        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p.e4m3 + row * p.C + blk * 32),
                     "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
        p.scales[fb4dev::mx_scale_offset(row, blk, nblk, p.scale_col_tiles, p.scale_tiled)] = (uint8_t)(Ech[0] - 3u);
      }
    } else if (active) {
      *reinterpret_cast<uint4*>(p.codes + row * code_row_bytes + blk * 16) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
      if (B16)   // two records
        *reinterpret_cast<uint32_t*>(p.meta + (row * nblk + blk) * 2) =
            ((Ech[0] - 3u) | ((uint32_t)didh[0] << 8)) | (((Ech[1] - 3u) | ((uint32_t)didh[1] << 8)) << 16);
      else
        p.meta[row * nblk + blk] = (uint16_t)((Ech[0] - 3u) | ((uint32_t)didh[0] << 8));
    }
    if (DECOMP) {
      int64_t srow = -1;
      while (list_next < cur.row) {
        ++list_pos;
        list_next = list_pos < ex.n_salient ? ex.salient_idx[list_pos] : 0x7fffffff;
      }
      if (list_next == cur.row) srow = list_pos;
      if (srow >= 0) {   // warp-uniform: a tile lies inside one token
        uint32_t rcw[4], rmeta;
        residual_block<SEDA, B16, CLAMP>(w, cw, didh, Ech, allowed, tb, qerr_base, pair_base, p.ec_lo, p.ec_hi, rcw,
                                         &rmeta);
        if (MX) {
          // the residual block as e4m3 bytes + E8M0 scale, row srow of the residual operand
          if (active) {
            const uint2 fb = tb->fb_e4m3[(rmeta >> 8) & 31u];
            uint32_t o[8];
#pragma unroll
            for (int q = 0; q < 4; ++q) fb4dev::codes_to_e4m3(rcw[q], fb, o[2 * q], o[2 * q + 1]);
            asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p.res_e4m3 + srow * p.C + blk * 32),
                         "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
            p.res_scales[fb4dev::mx_scale_offset(srow, blk, nblk, p.scale_col_tiles, p.scale_tiled)] = (uint8_t)rmeta;
          }
        } else if (active) {
          *reinterpret_cast<uint4*>(ex.res_codes + srow * code_row_bytes + blk * 16) =
              make_uint4(rcw[0], rcw[1], rcw[2], rcw[3]);
          if (B16) *reinterpret_cast<uint32_t*>(ex.res_meta + (srow * nblk + blk) * 2) = rmeta;
          else ex.res_meta[srow * nblk + blk] = (uint16_t)rmeta;
        }
      }
    }
    // ---- refill this stage (all lanes have consumed their registers from it)
    __syncwarp();
    if (lane == 0 && it_pre < n_mine) {
      mbar_expect_tx(bar, kTileBytes);
      tma_load_tile(my_ring + s * kTileBytes, &tmap, bar, pre.col * 16, pre.row);
    }
    ++it_pre;
    pre.advance(p, tpr);
    cur.advance(p, tpr);
#pragma unroll
    for (int k = 0; k + 1 < kStages; ++k) {
      cidq[k] = cidq[k + 1];
    }
    cidq[kStages - 1] = cid_new;
    maskq[0] = maskq[1];
    maskq[1] = mask_new;
    if (++s == kStages) { s = 0; parity ^= 1u; }
  }
  if (SEDA && bad_cid && lane == 0) atomicOr(p.status, 2u);
}

// ---------------------------------------------------------------------------------------------
// Contiguous tensors (ld == C): the tensor is one run of 32-element units and a tile is a run of
// consecutive units, whatever token they belong to, so every output address is linear in the unit
// number and the per-tile bookkeeping of the row / column walk is gone (2-D view [N/64][64] for TMA).
//  * Calls without a residual pass and with FB4 output: tiles of 4 KB = 64 units, two stages per warp;
//    lane i owns units 2i and 2i+1 (128 contiguous bytes = row i of the stage under the 128-byte
//    swizzle, eight conflict-free 16-byte shared loads).  One TMA load, one mbarrier wait, one 32-byte
//    code store and one 4-byte metadata store per lane serve two blocks.
//  * Calls with a residual pass or MXFP8 output: tiles of 2 KB = 32 units, four stages, lane i owns
//    unit i (half a row of the stage) - the register budget of the residual pass, and 32-byte e4m3
//    stores that cover whole lines, ask for one unit per lane.
// Token-dependent state (SeDA mask, salient list, tiled scale layout) follows a per-lane
// (token, unit-in-token) position; C is a multiple of 64, so the units 2i and 2i+1 share their token.
// The stage loop is unrolled, so stage addresses are immediates.  With block size 16 a unit is two blocks.
// units per lane and tile of a flat kernel
__host__ __device__ constexpr int flat_units(bool decomp, bool mx) { return (decomp || mx) ? 1 : 2; }

// NW warps per CTA: 16, or 20 for the kernels with a residual pass that fit 96 registers (three stages per warp then).
template <bool SEDA, bool DECOMP, bool B16, bool CLAMP, bool MX = false, int SEL = 0, int NW = kWarps>
__global__ void __launch_bounds__(NW * 32, 1)
fb4_quantize_flat_kernel(const __grid_constant__ CUtensorMap tmap, const SmemTables* __restrict__ g_tables,
                         FlatParams p, Fb4RowExtras ex) {
  constexpr int U = flat_units(DECOMP, MX);     // units per lane
  constexpr int kSt = NW == kWarps ? kStages / U : 3;   // stages per warp: 8 KB of ring per warp with 16 warps, 6 KB with 20
  constexpr int kRing = kSt * kTileBytes * U;           // ring bytes per warp
  constexpr int kTileB = kTileBytes * U;
  // which form the block routine's protection against non-finite input takes (by measurement: the branch costs
  // nothing where a lane holds two blocks, and less than the switchable loads in the MXFP8 kernel with a residual pass)
  constexpr bool kBranchy = U == 2 || (MX && DECOMP);
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* ring = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  SmemTables* tb = reinterpret_cast<SmemTables*>(ring + NW * kRing);
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(tb) + sizeof(SmemTables));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Tile -> warp assignment as in the strided kernel: interleaved over all warps of the grid, or (with a
  // residual pass) a contiguous range per CTA dealt round-robin to its warps.
  uint32_t g0, g_end, wstride;
  if (DECOMP) {
    const uint32_t per = p.n_tiles / gridDim.x, extra = p.n_tiles % gridDim.x, b = blockIdx.x;
    const uint32_t t0 = b * per + (b < extra ? b : extra);
    g0 = t0 + warp;
    g_end = t0 + per + (b < extra ? 1u : 0u);
    wstride = NW;
  } else {
    g0 = blockIdx.x * NW + warp;
    g_end = p.n_tiles;
    wstride = gridDim.x * NW;
  }
  const uint32_t table_bar = smem_u32(bars + NW * kStages);
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
  const uint32_t my_ring = smem_u32(ring + (size_t)warp * kRing);
  const uint32_t my_bars = smem_u32(bars + warp * kStages);
  const int32_t n_mine = g0 < g_end ? (int32_t)((g_end - g0 + wstride - 1) / wstride) : 0;
  int32_t y_pre = (int32_t)(g0 * (16u * U));      // first 128-byte row of the next tile to request
  const int32_t y_step = (int32_t)(wstride * (16u * U));
#pragma unroll
  for (int s = 0; s < kSt; ++s) {
    if (s < n_mine && lane == 0) {
      mbar_expect_tx(my_bars + 8 * s, kTileB);
      tma_load_2d(my_ring + s * kTileB, &tmap, my_bars + 8 * s, 0, y_pre);
    }
    y_pre += y_step;
  }
  // this lane's first unit of the current tile, and (where a token-dependent input or layout needs it)
  // the token / unit-in-token it falls in
  constexpr bool kNeedPos = SEDA || DECOMP || MX;
  uint32_t unit = g0 * (32u * U) + (uint32_t)(U * lane);
  const uint32_t unit_step = wstride * (32u * U);
  FlatPos pos{0, 0};
  if (kNeedPos) {
    pos.row = (int32_t)(unit / p.units_row);
    pos.rem = unit - (uint32_t)pos.row * p.units_row;
  }
  // SeDA: the cluster id of a lane's token is fetched three tiles ahead, its mask two tiles ahead.  Where the
  // value of a mask is first touched was settled by measurement: kernels with a residual pass run close to
  // their issue limit and must not wait for the mask when it is requested (the zero check waits for the use);
  // the others have slack there, and holding two more loads in flight across tiles cost them 3 to 5 %.
  constexpr bool kDeferMask = DECOMP;
  const bool use_seda = SEDA && ex.cluster_id != nullptr;
  const uint32_t n_cl = (uint32_t)ex.n_clusters;
  bool bad_cid = false;
  auto mask_of = [&](int32_t cid) -> uint32_t {
    if ((uint32_t)cid < n_cl) {
      const uint32_t m = ldg_early(ex.cluster_mask + cid);
      return kDeferMask ? m : (m ? m : 1u);   // a zero mask (precondition violated) yields dialect 0: stay in bounds
    }
    if (cid != -1) bad_cid = true;  // outside [-1, n_clusters): unconstrained, reported in bit 1 of the status word
    return 0xffffffffu;
  };
  uint32_t mask_cur = 0xffffffffu, mask_nx = 0xffffffffu;
  int32_t cid_n2 = -1;
  FlatPos pos_pf = pos;
  uint32_t unit_pf = unit;
  if (SEDA) {
    if (use_seda) {
      auto cid_at = [&](int k) -> int32_t { return (k < n_mine && unit_pf < p.n_units) ? (int32_t)ldg_early(ex.cluster_id + pos_pf.row) : -1; };
      mask_cur = mask_of(cid_at(0));
      pos_pf.advance(p); unit_pf += unit_step;
      mask_nx = mask_of(cid_at(1));
      pos_pf.advance(p); unit_pf += unit_step;
      cid_n2 = cid_at(2);
      pos_pf.advance(p); unit_pf += unit_step;
    }
  }
  // salient tokens: an ascending list; a lane's tokens never decrease, so a cursor walks it
  int64_t list_pos = 0;
  int32_t list_next = 0x7fffffff;
  if (DECOMP && n_mine > 0) {
    int64_t lo = 0, hi = ex.n_salient;
    while (lo < hi) {
      const int64_t mid = (lo + hi) >> 1;
      if (ex.salient_idx[mid] < pos.row) lo = mid + 1; else hi = mid;
    }
    list_pos = lo;
    if (lo < ex.n_salient) list_next = ex.salient_idx[lo];
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
  // this lane's 16-byte chunks in stage 0.  Two units: row `lane` of 128 B, chunk j at position j ^ (lane & 7).
  // One unit: row lane / 2, chunks (lane & 1) * 4 + j.
  uint32_t chunk[4 * U];
#pragma unroll
  for (int j = 0; j < 4 * U; ++j) {
    const uint32_t r = U == 2 ? (uint32_t)lane : ((uint32_t)lane >> 1);
    const uint32_t c = U == 2 ? (uint32_t)j : (((uint32_t)lane & 1u) * 4u + (uint32_t)j);
    chunk[j] = my_ring + r * 128u + ((c ^ (r & 7u)) << 4);
  }

  // The stage loop is unrolled (stage addresses become immediates) except with a residual pass, whose
  // body is too long to be worth several copies (measured: 0.38 ms against 0.39 and 0.42 ms for two and four).
  constexpr int kUnroll = DECOMP ? 1 : kSt;
  uint32_t parity = 0;
  int s_dyn = 0;
  bool failed = false;
  for (int32_t it = 0; it < n_mine && !failed; it += kUnroll) {
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int s = kUnroll == kSt ? u : s_dyn;
      if (it + u < n_mine && !failed) {
        // ---- SeDA inputs of the tiles ahead
        uint32_t mask_new = 0xffffffffu;
        int32_t cid_new = -1;
        if (SEDA) {
          if (use_seda) {
            mask_new = mask_of(cid_n2);
            if (it + u + 3 < n_mine && unit_pf < p.n_units) cid_new = (int32_t)ldg_early(ex.cluster_id + pos_pf.row);
            pos_pf.advance(p);
            unit_pf += unit_step;
          }
        }
        const uint32_t bar = my_bars + 8 * s;
        uint32_t spins = 0;
        bool ready = mbar_try_wait(bar, parity);
        while (!ready && ++spins < kSpinLimit) ready = mbar_try_wait(bar, parity);
        if (!__all_sync(0xffffffffu, ready)) {
          // A load never arrived: raise the status bit, give the loads still in flight for this warp a
          // bounded chance to land (so none writes into shared memory after the CTA has gone), stop.
          if (lane == 0) atomicOr(p.status, 1u);
          for (int j = 1; j < kSt; ++j) {
            if (it + u + j >= n_mine) break;
            const int sj = (s + j) % kSt;
            const uint32_t pj = (s + j) >= kSt ? (parity ^ 1u) : parity;
            uint32_t tries = 0;
            while (!mbar_try_wait(my_bars + 8 * sj, pj) && ++tries < kSpinLimit) {}
          }
          failed = true;
        } else {
          const bool active = unit < p.n_units;
          const uint32_t allowed = SEDA ? (kDeferMask ? (mask_cur ? mask_cur : 1u) : mask_cur) : 0xffffffffu;
          int64_t srow = -1;
          if (DECOMP) {
            while (list_next < pos.row) {
              ++list_pos;
              list_next = list_pos < ex.n_salient ? ex.salient_idx[list_pos] : 0x7fffffff;
            }
            if (list_next == pos.row && active) srow = list_pos;
          }
          uint32_t cw[4 * U], mrec[U];      // per unit: code words, metadata (one record, or two with block size 16)
          int did0[U];
#pragma unroll
          for (int h = 0; h < U; ++h) {
            uint32_t w[16];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint4 v = lds_v4(chunk[4 * h + j] + s * kTileB);
              w[4 * j] = v.x; w[4 * j + 1] = v.y; w[4 * j + 2] = v.z; w[4 * j + 3] = v.w;
            }
            uint32_t c4[4], Ech[2];
            int didh[2];
            quantize_packed_block<SEDA, B16, CLAMP, SEL, kBranchy>(w, allowed, tb, qerr_base, pair_base, p.ec_lo, p.ec_hi, c4,
                                                                   didh, Ech);
#pragma unroll
            for (int q = 0; q < 4; ++q) cw[4 * h + q] = c4[q];
            did0[h] = didh[0];
            mrec[h] = B16 ? (((Ech[0] - 3u) | ((uint32_t)didh[0] << 8)) | (((Ech[1] - 3u) | ((uint32_t)didh[1] << 8)) << 16))
                          : ((Ech[0] - 3u) | ((uint32_t)didh[0] << 8));
            if (DECOMP) {     // one unit per lane: the residual follows at once, from the same registers
              if (srow >= 0) {
                uint32_t rcw[4], rrec;
                residual_block<SEDA, B16, CLAMP, SEL, kBranchy>(w, c4, didh, Ech, allowed, tb, qerr_base, pair_base, p.ec_lo, p.ec_hi,
                                                 rcw, &rrec);
                const size_t ru = (size_t)srow * p.units_row + pos.rem;      // unit of the residual tensor
                if (MX) {
                  const uint2 fb = tb->fb_e4m3[(rrec >> 8) & 31u];
                  uint32_t o[8];
#pragma unroll
                  for (int q = 0; q < 4; ++q) fb4dev::codes_to_e4m3(rcw[q], fb, o[2 * q], o[2 * q + 1]);
                  stg_v8(p.res_e4m3 + ru * 32u, o);
                  p.res_scales[fb4dev::mx_scale_offset(srow, pos.rem, p.units_row, p.scale_col_tiles, p.scale_tiled)] =
                      (uint8_t)rrec;
                } else {
                  *reinterpret_cast<uint4*>(ex.res_codes + ru * 16u) = make_uint4(rcw[0], rcw[1], rcw[2], rcw[3]);
                  if (B16) *reinterpret_cast<uint32_t*>(ex.res_meta + ru * 2u) = rrec;
                  else ex.res_meta[ru] = (uint16_t)rrec;
                }
              }
            }
          }
          if (active) {
            if (MX) {
              // the codes become e4m3 bytes in registers, 32 contiguous bytes per lane; the scale byte is the E8M0 scale
              const uint2 fb = tb->fb_e4m3[did0[0]];
              uint32_t o[8];
#pragma unroll
              for (int q = 0; q < 4; ++q) fb4dev::codes_to_e4m3(cw[q], fb, o[2 * q], o[2 * q + 1]);
              stg_v8(p.e4m3 + (size_t)unit * 32u, o);
              const int64_t so = p.scale_tiled ? fb4dev::mx_scale_offset(pos.row, pos.rem, p.units_row, p.scale_col_tiles, 1)
                                               : (int64_t)unit;
              p.scales[so] = (uint8_t)mrec[0];
            } else if (U == 2) {
              stg_v8(p.codes + (size_t)unit * 16u, cw);
              if (B16) *reinterpret_cast<uint2*>(p.meta + (size_t)unit * 2u) = make_uint2(mrec[0], mrec[U - 1]);
              else *reinterpret_cast<uint32_t*>(p.meta + unit) = mrec[0] | (mrec[U - 1] << 16);
            } else {
              *reinterpret_cast<uint4*>(p.codes + (size_t)unit * 16u) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
              if (B16) *reinterpret_cast<uint32_t*>(p.meta + (size_t)unit * 2u) = mrec[0];
              else p.meta[unit] = (uint16_t)mrec[0];
            }
          }
          // ---- refill this stage (all lanes have consumed their registers from it)
          __syncwarp();
          if (lane == 0 && it + u + kSt < n_mine) {
            mbar_expect_tx(bar, kTileB);
            tma_load_2d(my_ring + s * kTileB, &tmap, bar, 0, y_pre);
          }
          y_pre += y_step;
          unit += unit_step;
          if (kNeedPos) pos.advance(p);
          if (SEDA) {
            mask_cur = mask_nx;
            mask_nx = mask_new;
            cid_n2 = cid_new;
          }
        }
      }
    }
    if (kUnroll == kSt) {
      parity ^= 1u;
    } else if (++s_dyn == kSt) {
      s_dyn = 0;
      parity ^= 1u;
    }
  }
  if (SEDA && bad_cid) atomicOr(p.status, 2u);
}


// ---------------------------------------------------------------------------------------------
// fp32 input (the hook for a producer that still holds its result in fp32): same ring and tables,
// 16 warps per CTA, tiles of 1024 channels = 4 KB (view [T][C/32][32 floats], box 1 x 32 x 32,
// 128-byte swizzle: row r of a stage is block r).  Lane i reads its block with eight conflict-free
// 16-byte shared loads, keeps the upper 16 bits of every value and quantizes them with
// quantize_packed_block.
constexpr int kWarpsF32 = 16;      // 80 registers; two stages of 4 KB each keep the ring at 128 KB
constexpr int kStagesF32 = 2;
constexpr int kTileBytesF32 = 4096;

__global__ void __launch_bounds__(kWarpsF32 * 32, 1)
fb4_quantize_f32_kernel(const __grid_constant__ CUtensorMap tmap, const SmemTables* __restrict__ g_tables,
                        FastParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* ring = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  SmemTables* tb = reinterpret_cast<SmemTables*>(ring + kWarpsF32 * kStagesF32 * kTileBytesF32);
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(tb) + sizeof(SmemTables));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t gwarp = (int64_t)blockIdx.x * kWarpsF32 + warp;
  const int64_t wstride = (int64_t)gridDim.x * kWarpsF32;
  const int32_t tpr = (int32_t)p.tiles_per_row;

  const uint32_t table_bar = smem_u32(bars + kWarpsF32 * kStagesF32);
  // every warp initialises its own ring barriers; the first thread also the table barrier, and it
  // starts the table copy at once (one thread doing all kWarpsF32 * kStagesF32 + 1 inits in a row used to
  // hold the whole CTA for most of a microsecond)
  if (lane == 0) {
    for (int i = 0; i < kStagesF32; ++i) mbar_init(smem_u32(bars + warp * kStagesF32 + i), 1);
    if (warp == 0) mbar_init(table_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (warp == 0) {
      mbar_expect_tx(table_bar, (uint32_t)sizeof(SmemTables));
      bulk_load(smem_u32(tb), g_tables, (uint32_t)sizeof(SmemTables), table_bar);
    }
  }
  __syncthreads();

  const uint32_t my_ring = smem_u32(ring + (size_t)warp * kStagesF32 * kTileBytesF32);
  const uint32_t my_bars = smem_u32(bars + warp * kStagesF32);
  TilePos cur, pre;
  cur.row = (int32_t)(gwarp / tpr);
  cur.col = (int32_t)(gwarp - (int64_t)cur.row * tpr);
  pre = cur;
  const int32_t n_mine = gwarp < p.n_tiles ? (int32_t)((p.n_tiles - gwarp + wstride - 1) / wstride) : 0;
  int32_t it_pre = 0;
#pragma unroll
  for (int s = 0; s < kStagesF32; ++s) {
    if (it_pre < n_mine && lane == 0) {
      mbar_expect_tx(my_bars + 8 * s, kTileBytesF32);
      tma_load_tile(my_ring + s * kTileBytesF32, &tmap, my_bars + 8 * s, pre.col * 32, pre.row);
    }
    ++it_pre;
    pre.advance(p, tpr);
  }
  {
    uint32_t spins = 0;
    bool ready = mbar_try_wait(table_bar, 0u);
    while (!ready && ++spins < kSpinLimit) ready = mbar_try_wait(table_bar, 0u);
    if (!__all_sync(0xffffffffu, ready)) {
      if (lane == 0) atomicOr(p.status, 1u);
      for (int j = 0; j < kStagesF32 && j < n_mine; ++j) {
        uint32_t tries = 0;
        while (!mbar_try_wait(my_bars + 8 * j, 0u) && ++tries < kSpinLimit) {}
      }
      return;
    }
  }
  const uint32_t pair_base = smem_u32(tb->pairlut);
  const uint32_t qerr_base = smem_u32(tb->qerr_private) + ((uint32_t)lane & 15u) * 8u;
  uint32_t chunk_off[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) chunk_off[j] = (uint32_t)lane * 128u + ((((uint32_t)j) ^ ((uint32_t)lane & 7u)) << 4);
  const int64_t nblk = p.C >> 5;
  const int64_t code_row_bytes = p.C >> 1;

  int s = 0;
  uint32_t parity = 0;
  for (int32_t it = 0; it < n_mine; ++it) {
    const uint32_t bar = my_bars + 8 * s;
    uint32_t spins = 0;
    bool ready = mbar_try_wait(bar, parity);
    while (!ready && ++spins < kSpinLimit) ready = mbar_try_wait(bar, parity);
    if (!__all_sync(0xffffffffu, ready)) {
      if (lane == 0) atomicOr(p.status, 1u);
      int sj = s;
      uint32_t pj = parity;
      for (int j = 1; j < kStagesF32; ++j) {
        if (it + j >= n_mine) break;
        if (++sj == kStagesF32) { sj = 0; pj ^= 1u; }
        uint32_t tries = 0;
        while (!mbar_try_wait(my_bars + 8 * sj, pj) && ++tries < kSpinLimit) {}
      }
      break;
    }
    const int64_t row = cur.row;
    const int64_t blk = (int64_t)cur.col * 32 + lane;
    uint32_t xw[16];   // the upper 16 bits of every value, two per register (all the quantizer needs)
    {
      const uint32_t base = my_ring + s * kTileBytesF32;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint4 v0 = lds_v4(base + chunk_off[2 * q]), v1 = lds_v4(base + chunk_off[2 * q + 1]);
        xw[4 * q] = __byte_perm(v0.x, v0.y, 0x7632);
        xw[4 * q + 1] = __byte_perm(v0.z, v0.w, 0x7632);
        xw[4 * q + 2] = __byte_perm(v1.x, v1.y, 0x7632);
        xw[4 * q + 3] = __byte_perm(v1.z, v1.w, 0x7632);
      }
    }
    uint32_t cw[4], Eb[2];
    int did[2];
    quantize_packed_block<false, false, false>(xw, 0xffffffffu, tb, qerr_base, pair_base, 3u, 254u, cw, did, Eb);
    const uint32_t m = (Eb[0] - 3u) | ((uint32_t)did[0] << 8);
    if (blk < nblk) {
      *reinterpret_cast<uint4*>(p.codes + row * code_row_bytes + blk * 16) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
      p.meta[row * nblk + blk] = (uint16_t)m;
    }
    __syncwarp();
    if (lane == 0 && it_pre < n_mine) {
      mbar_expect_tx(bar, kTileBytesF32);
      tma_load_tile(my_ring + s * kTileBytesF32, &tmap, bar, pre.col * 32, pre.row);
    }
    ++it_pre;
    pre.advance(p, tpr);
    cur.advance(p, tpr);
    if (++s == kStagesF32) { s = 0; parity ^= 1u; }
  }
}

constexpr size_t kSmemBytesF32 =
    1024 + (size_t)kWarpsF32 * kStagesF32 * kTileBytesF32 + sizeof(SmemTables) + (kWarpsF32 * kStagesF32 + 1) * 8;
static_assert(kSmemBytesF32 <= 227 * 1024, "shared memory budget of one CTA");

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up once (safe from several host threads).
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

constexpr int kWarpsWide = 20;
constexpr size_t kSmemBytesWide =
    1024 + (size_t)kWarpsWide * 3 * kTileBytes + sizeof(SmemTables) + (kWarpsWide * kStages + 1) * 8;
static_assert(kSmemBytesWide <= 227 * 1024, "shared memory budget of one CTA");

template <bool SEDA, bool DECOMP, bool B16, bool CLAMP>
cudaError_t launch(const CUtensorMap& map, const SmemTables* tables, const FastParams& p, const Fb4RowExtras& ex,
                   int grid, cudaStream_t stream) {
  fb4_quantize_fast_kernel<SEDA, DECOMP, B16, CLAMP><<<grid, kWarps * 32, kSmemBytes, stream>>>(map, tables, p, ex);
  return cudaGetLastError();
}

}  // namespace

// Builds the packed tables of this kernel from the plain ones; returns false when the formatbook /
// stage-1 table does not fit them (more than 8 groups, a group with 0 or more than 8 dialects, or
// error sums that could overflow a byte): those contexts use the generic kernel.
bool fb4_fast_build_tables(const Fb4DeviceTables& t, int select_mode, void** d_out, size_t* bytes) {
  FastTables ft;
  std::memset(&ft, 0, sizeof ft);
  uint32_t groups[kMaxGroups];
  int ngroups = 0;
  // A context that scores every dialect never looks a stage-1 group up: its error words hold the 32 dialects
  // once, eight to a word in id order, instead of the (padded) stage-1 groups.
  if (select_mode == 1) {
    for (int i = 0; i < 4; ++i) groups[i] = 0xffu << (8 * i);
    ngroups = 4;
  }
  for (int k = 0; k < 32 && select_mode == 1; ++k) ft.stage1[k] = t.stage1[k];
  for (int k = 0; k < 32 && select_mode != 1; ++k) {
    const uint32_t m = t.stage1[k];
    const int pc = __builtin_popcount(m);
    if (pc == 0 || pc > 8) return false;
    int gi = -1;
    for (int i = 0; i < ngroups; ++i) if (groups[i] == m) gi = i;
    if (gi < 0) {
      if (ngroups == kMaxGroups) return false;
      gi = ngroups;
      groups[ngroups++] = m;
    }
    ft.group_of_bin[k] = (uint8_t)gi;
    ft.stage1[k] = m;
  }
  for (int gi = 0; gi < ngroups; ++gi) {
    int j = 0;
    for (int d = 0; d < 32; ++d) {
      if (!((groups[gi] >> d) & 1u)) continue;
      ft.did_of[gi][j] = (uint8_t)d;
      for (int k = 0; k < 32; ++k) {
        if (t.qerror[d][k] > 31) return false;
        ft.qerr64[gi][k] |= (uint64_t)t.qerror[d][k] << (8 * j);
      }
      ++j;
    }
    for (; j < 8; ++j)
      for (int k = 0; k < 32; ++k) ft.qerr64[gi][k] |= (uint64_t)31 << (8 * j);   // never beats a real candidate
  }
  ft.n_groups = (uint32_t)ngroups;
  for (int gi = 0; gi < kMaxGroups; ++gi) {
    uint32_t id[8];
    for (int j = 0; j < 8; ++j) id[j] = (gi < ngroups && j < __builtin_popcount(groups[gi])) ? ft.did_of[gi][j] : 31u;
    ft.did_lanes[gi] = make_uint4(id[0] | (id[2] << 16), id[1] | (id[3] << 16), id[4] | (id[6] << 16), id[5] | (id[7] << 16));
  }
  std::memcpy(ft.qvalue, t.qvalue, sizeof ft.qvalue);
  std::memcpy(ft.qerror, t.qerror, sizeof ft.qerror);
  std::memcpy(ft.fb, t.formatbook, sizeof ft.fb);
  // the image every CTA copies into its shared memory
  SmemTables* img = new (std::nothrow) SmemTables;
  if (!img) return false;
  std::memset(img, 0, sizeof *img);
  for (int g = 0; g < kMaxGroups; ++g)
    for (int k = 0; k < 32; ++k)
      for (int c = 0; c < 16; ++c) img->qerr_private[g][k][c] = ft.qerr64[g][k];
  for (int d = 0; d < 32; ++d)
    for (int bh = 0; bh < 32; ++bh)
      for (int bl = 0; bl < 32; ++bl)
        img->pairlut[d * kPairStride + bh * kPairMul + bl] = (uint8_t)(t.qvalue[d][bl] | (t.qvalue[d][bh] << 4));
  for (int d = 0; d < 32; ++d) {
    uint8_t* row = reinterpret_cast<uint8_t*>(&img->fb_bf16[d]);
    for (int j = 0; j < 8; ++j) {
      const float f = (float)t.formatbook[d][j];   // integers 0..15 are exact in bf16
      uint32_t u;
      std::memcpy(&u, &f, 4);
      row[j] = (uint8_t)(u >> 24);
      row[8 + j] = (uint8_t)(u >> 16);
    }
  }
  for (int d = 0; d < 32; ++d)
    for (int j = 0; j < 8; ++j)
      reinterpret_cast<uint8_t*>(&img->fb_e4m3[d])[j] = (uint8_t)fb4dev::e4m3_of_small_int(t.formatbook[d][j]);
  img->c = ft;
  void* d = nullptr;
  bool ok = cudaMalloc(&d, sizeof *img) == cudaSuccess;
  if (ok && cudaMemcpy(d, img, sizeof *img, cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaFree(d);
    ok = false;
  }
  delete img;
  if (!ok) return false;
  *d_out = d;
  *bytes = sizeof(SmemTables);
  return true;
}

// Opt in to the kernel's dynamic shared memory on the current device (once per context).
cudaError_t fb4_fast_prepare_device() {
  const int bytes = (int)kSmemBytes;
  const cudaFuncAttribute attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
  cudaError_t e = cudaSuccess;
#define FB4_OPT_IN(...) \
  if (e == cudaSuccess) e = cudaFuncSetAttribute(fb4_quantize_fast_kernel<__VA_ARGS__>, attr, bytes)
  FB4_OPT_IN(false, false, false, false);
  FB4_OPT_IN(true, false, false, false);
  FB4_OPT_IN(false, true, false, false);
  FB4_OPT_IN(true, true, false, false);
  FB4_OPT_IN(false, false, true, false);
  FB4_OPT_IN(true, false, true, false);
  FB4_OPT_IN(false, true, true, false);
  FB4_OPT_IN(true, true, true, false);
  FB4_OPT_IN(false, false, false, true);
  FB4_OPT_IN(true, false, false, true);
  FB4_OPT_IN(false, true, false, true);
  FB4_OPT_IN(true, true, false, true);
  FB4_OPT_IN(false, false, true, true);
  FB4_OPT_IN(true, false, true, true);
  FB4_OPT_IN(false, true, true, true);
  FB4_OPT_IN(true, true, true, true);
  FB4_OPT_IN(false, false, false, false, true);
  FB4_OPT_IN(true, false, false, false, true);
  FB4_OPT_IN(false, true, false, false, true);
  FB4_OPT_IN(true, true, false, false, true);
#undef FB4_OPT_IN
#define FB4_OPT_IN(...) \
  if (e == cudaSuccess) e = cudaFuncSetAttribute(fb4_quantize_flat_kernel<__VA_ARGS__>, attr, (int)kSmemBytes)
  FB4_OPT_IN(false, false, false, false);
  FB4_OPT_IN(true, false, false, false);
  FB4_OPT_IN(false, true, false, false);
  FB4_OPT_IN(true, true, false, false);
  FB4_OPT_IN(false, false, true, false);
  FB4_OPT_IN(true, false, true, false);
  FB4_OPT_IN(false, true, true, false);
  FB4_OPT_IN(true, true, true, false);
  FB4_OPT_IN(false, false, false, true);
  FB4_OPT_IN(true, false, false, true);
  FB4_OPT_IN(false, true, false, true);
  FB4_OPT_IN(true, true, false, true);
  FB4_OPT_IN(false, false, true, true);
  FB4_OPT_IN(true, false, true, true);
  FB4_OPT_IN(false, true, true, true);
  FB4_OPT_IN(true, true, true, true);
  FB4_OPT_IN(false, false, false, false, true);
  FB4_OPT_IN(true, false, false, false, true);
  FB4_OPT_IN(false, true, false, false, true);
  FB4_OPT_IN(true, true, false, false, true);
  FB4_OPT_IN(false, false, false, false, false, 1);
  FB4_OPT_IN(true, false, false, false, false, 1);
  FB4_OPT_IN(false, true, false, false, false, 1);
  FB4_OPT_IN(true, true, false, false, false, 1);
  FB4_OPT_IN(false, false, false, false, false, 2);
  FB4_OPT_IN(true, false, false, false, false, 2);
  FB4_OPT_IN(false, true, false, false, false, 2);
  FB4_OPT_IN(true, true, false, false, false, 2);
#undef FB4_OPT_IN
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(fb4_quantize_flat_kernel<false, true, false, false, false, 0, kWarpsWide>, attr, (int)kSmemBytesWide);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(fb4_quantize_flat_kernel<true, true, false, false, false, 0, kWarpsWide>, attr, (int)kSmemBytesWide);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(fb4_quantize_f32_kernel, attr, (int)kSmemBytesF32);
  if (e == cudaSuccess) e = fb4_producers_prepare_device();
  return e;
}

// Block sizes 32 and 16, any exponent clamp (the 5-bit exponent of Sec. 3.1 included), every
// extension; num_groups 8 and two-stage selection only.
bool fb4_fast_eligible(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld) {
  const fb4_config& c = ctx->cfg;
  if (!ctx->fast_ok || !ctx->d_fast_tables) return false;
  if (c.block_size != 32 && c.block_size != 16) return false;
  if (c.num_groups != 8 || c.select_mode != 0) {
    // every element its own group, or every dialect scored: block size 32, full exponent range, contiguous rows
    const bool per_element = c.num_groups == 32 && c.select_mode == 0, all = c.num_groups == 8 && c.select_mode == 1;
    if (!(per_element || all) || c.block_size != 32 || c.exp_min != -124 || c.exp_max != 127 || ld != C) return false;
    if (T <= 0 || T * (C / 32) >= 0x7fffffffLL) return false;   // these modes exist in the kernel for contiguous tensors only
  }
  if (C % 64 != 0 || (ld & 7) || (reinterpret_cast<uintptr_t>(x) & 15)) return false;
  if (T > 0x7fffffffLL || C / 64 > 0x7fffffffLL) return false;
  return encode_tiled_fn() != nullptr;
}

static_assert(sizeof(CUtensorMap) == sizeof(Fb4TensorMapSlot::map), "slot size");

// The encoded tensor map of (x, T, C, ld) for kernel family `kind`: from the context's slot if the last launch
// of that family had the same arguments, else encoded by `encode` and kept.
template <typename Encode>
static cudaError_t cached_tensor_map(const fb4_ctx* ctx, int kind, const void* x, int64_t T, int64_t C, int64_t ld,
                                     CUtensorMap* map, Encode encode) {
  Fb4TensorMapSlot& sl = ctx->tmap_slot[kind];
  if (sl.valid && sl.x == x && sl.T == T && sl.C == C && sl.ld == ld) {
    std::memcpy(map, sl.map, sizeof(CUtensorMap));
    return cudaSuccess;
  }
  if (encode(map) != CUDA_SUCCESS) return cudaErrorInvalidValue;
  sl.x = x; sl.T = T; sl.C = C; sl.ld = ld;
  std::memcpy(sl.map, map, sizeof(CUtensorMap));
  sl.valid = 1;
  return cudaSuccess;
}

// Tensor map, grid and tile-walk parameters of one launch of the bf16-input kernels.
static cudaError_t fast_setup(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, bool chunked,
                              CUtensorMap* map, FastParams* p, int* grid_out) {
  const cuuint64_t dims[3] = {64, (cuuint64_t)(C / 64), (cuuint64_t)T};
  const cuuint64_t strides[2] = {128, (cuuint64_t)ld * 2};
  const cuuint32_t box[3] = {64, 16, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const cudaError_t ce = cached_tensor_map(ctx, 0, x, T, C, ld, map, [&](CUtensorMap* m) {
    return encode_tiled_fn()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(x), dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  });
  if (ce != cudaSuccess) return ce;
  *p = FastParams{};
  p->T = T;
  p->C = C;
  p->tiles_per_row = (C + 1023) / 1024;
  p->n_tiles = T * p->tiles_per_row;
  p->status = ctx->d_status;
  const int64_t want = (p->n_tiles + kWarps - 1) / kWarps;
  const int grid = (int)(want < ctx->sm_count ? want : ctx->sm_count);
  const int64_t wstride = chunked ? kWarps : (int64_t)grid * kWarps;   // tiles between a warp's consecutive tiles
  p->step_rows = wstride / p->tiles_per_row;
  p->step_cols = (int32_t)(wstride % p->tiles_per_row);
  p->ec_lo = (uint32_t)(ctx->cfg.exp_min + 127);
  p->ec_hi = (uint32_t)(ctx->cfg.exp_max + 127);
  *grid_out = grid;
  return cudaSuccess;
}

// The flat kernel takes contiguous tensors whose unit count fits 31 bits.
static bool flat_eligible(int64_t T, int64_t C, int64_t ld) {
  return ld == C && C % 64 == 0 && T > 0 && T * (C / 32) < 0x7fffffffLL;
}

// Tensor map (2-D view [N/64][64] of the contiguous tensor), grid and walk parameters of one flat launch.
static cudaError_t flat_setup(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, bool chunked, bool mx,
                              CUtensorMap* map, FlatParams* p, int* grid_out, int nw = kWarps) {
  const uint32_t U = (uint32_t)flat_units(chunked, mx);   // units per lane: tiles of 32 * U units = 2 KB * U
  const cuuint64_t dims[2] = {64, (cuuint64_t)(T * C / 64)};
  const cuuint64_t strides[1] = {128};
  const cuuint32_t box[2] = {64, 16 * U};
  const cuuint32_t estr[2] = {1, 1};
  const cudaError_t ce = cached_tensor_map(ctx, (int)U, x, T, C, C, map, [&](CUtensorMap* m) {
    return encode_tiled_fn()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(x), dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  });
  if (ce != cudaSuccess) return ce;
  *p = FlatParams{};
  p->units_row = (uint32_t)(C / 32);
  p->n_units = (uint32_t)(T * (C / 32));
  p->n_tiles = (p->n_units + 32u * U - 1u) / (32u * U);
  p->status = ctx->d_status;
  const int64_t want = ((int64_t)p->n_tiles + nw - 1) / nw;
  const int grid = (int)(want < ctx->sm_count ? want : ctx->sm_count);
  const uint64_t unit_step = (uint64_t)(chunked ? nw : grid * nw) * 32u * U;
  p->step_rows = (uint32_t)(unit_step / p->units_row);
  p->step_rem = (uint32_t)(unit_step % p->units_row);
  p->ec_lo = (uint32_t)(ctx->cfg.exp_min + 127);
  p->ec_hi = (uint32_t)(ctx->cfg.exp_max + 127);
  *grid_out = grid;
  return cudaSuccess;
}

template <bool SEDA, bool DECOMP, bool B16, bool CLAMP>
static cudaError_t launch_flat(const CUtensorMap& map, const SmemTables* tables, const FlatParams& p,
                               const Fb4RowExtras& ex, int grid, cudaStream_t stream) {
  fb4_quantize_flat_kernel<SEDA, DECOMP, B16, CLAMP><<<grid, kWarps * 32, kSmemBytes, stream>>>(map, tables, p, ex);
  return cudaGetLastError();
}

cudaError_t fb4_launch_quantize_fast(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld,
                                     const Fb4RowExtras& ex, uint8_t* codes, uint16_t* meta, cudaStream_t stream) {
  const bool seda = ex.cluster_id != nullptr, decomp = ex.n_salient > 0;
  CUtensorMap map;
  if (flat_eligible(T, C, ld)) {
    FlatParams fp;
    int grid = 0;
    const bool b16 = ctx->cfg.block_size == 16;
    const bool clamp = ctx->cfg.exp_min != -124 || ctx->cfg.exp_max != 127;
    const int sel = ctx->cfg.num_groups == 32 ? 1 : (ctx->cfg.select_mode == 1 ? 2 : 0);
    // the default configuration with a residual pass fits 96 registers: 20 warps per CTA
    const bool wide = decomp && !b16 && !clamp && sel == 0;
    const cudaError_t e = flat_setup(ctx, x, T, C, decomp, false, &map, &fp, &grid, wide ? kWarpsWide : kWarps);
    if (e != cudaSuccess) return e;
    fp.codes = codes;
    fp.meta = meta;
    const SmemTables* tables = static_cast<const SmemTables*>(ctx->d_fast_tables);
    if (wide) {
      if (seda)
        fb4_quantize_flat_kernel<true, true, false, false, false, 0, kWarpsWide>
            <<<grid, kWarpsWide * 32, kSmemBytesWide, stream>>>(map, tables, fp, ex);
      else
        fb4_quantize_flat_kernel<false, true, false, false, false, 0, kWarpsWide>
            <<<grid, kWarpsWide * 32, kSmemBytesWide, stream>>>(map, tables, fp, ex);
      return cudaGetLastError();
    }
    if (sel != 0) {
#define FB4_SEL(S, D, L) \
  fb4_quantize_flat_kernel<S, D, false, false, false, L><<<grid, kWarps * 32, kSmemBytes, stream>>>(map, tables, fp, ex)
      switch ((seda ? 1 : 0) | (decomp ? 2 : 0) | (sel == 2 ? 4 : 0)) {
        case 0: FB4_SEL(false, false, 1); break;
        case 1: FB4_SEL(true, false, 1); break;
        case 2: FB4_SEL(false, true, 1); break;
        case 3: FB4_SEL(true, true, 1); break;
        case 4: FB4_SEL(false, false, 2); break;
        case 5: FB4_SEL(true, false, 2); break;
        case 6: FB4_SEL(false, true, 2); break;
        default: FB4_SEL(true, true, 2); break;
      }
#undef FB4_SEL
      return cudaGetLastError();
    }
    switch ((seda ? 1 : 0) | (decomp ? 2 : 0) | (b16 ? 4 : 0) | (clamp ? 8 : 0)) {
#define FB4_CASE(V, S, D, B, K) \
  case V: return launch_flat<S, D, B, K>(map, tables, fp, ex, grid, stream)
      FB4_CASE(0, false, false, false, false);
      FB4_CASE(1, true, false, false, false);
      FB4_CASE(2, false, true, false, false);
      FB4_CASE(3, true, true, false, false);
      FB4_CASE(4, false, false, true, false);
      FB4_CASE(5, true, false, true, false);
      FB4_CASE(6, false, true, true, false);
      FB4_CASE(7, true, true, true, false);
      FB4_CASE(8, false, false, false, true);
      FB4_CASE(9, true, false, false, true);
      FB4_CASE(10, false, true, false, true);
      FB4_CASE(11, true, true, false, true);
      FB4_CASE(12, false, false, true, true);
      FB4_CASE(13, true, false, true, true);
      FB4_CASE(14, false, true, true, true);
      FB4_CASE(15, true, true, true, true);
#undef FB4_CASE
    }
    return cudaErrorInvalidValue;
  }
  FastParams p;
  int grid = 0;
  const cudaError_t e = fast_setup(ctx, x, T, C, ld, decomp, &map, &p, &grid);
  if (e != cudaSuccess) return e;
  p.codes = codes;
  p.meta = meta;
  const SmemTables* tables = static_cast<const SmemTables*>(ctx->d_fast_tables);
  const bool b16 = ctx->cfg.block_size == 16;
  const bool clamp = ctx->cfg.exp_min != -124 || ctx->cfg.exp_max != 127;
  const int variant = (seda ? 1 : 0) | (decomp ? 2 : 0) | (b16 ? 4 : 0) | (clamp ? 8 : 0);
  switch (variant) {
#define FB4_CASE(V, S, D, B, K) \
  case V: return launch<S, D, B, K>(map, tables, p, ex, grid, stream)
    FB4_CASE(0, false, false, false, false);
    FB4_CASE(1, true, false, false, false);
    FB4_CASE(2, false, true, false, false);
    FB4_CASE(3, true, true, false, false);
    FB4_CASE(4, false, false, true, false);
    FB4_CASE(5, true, false, true, false);
    FB4_CASE(6, false, true, true, false);
    FB4_CASE(7, true, true, true, false);
    FB4_CASE(8, false, false, false, true);
    FB4_CASE(9, true, false, false, true);
    FB4_CASE(10, false, true, false, true);
    FB4_CASE(11, true, true, false, true);
    FB4_CASE(12, false, false, true, true);
    FB4_CASE(13, true, false, true, true);
    FB4_CASE(14, false, true, true, true);
    FB4_CASE(15, true, true, true, true);
#undef FB4_CASE
  }
  return cudaErrorInvalidValue;
}

bool fb4_fast_f32_eligible(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld) {
  const fb4_config& c = ctx->cfg;
  if (!ctx->fast_ok || !ctx->d_fast_tables) return false;
  if (c.block_size != 32 || c.num_groups != 8 || c.select_mode != 0 || c.exp_min != -124 || c.exp_max != 127)
    return false;
  if (C % 32 != 0 || (ld & 3) || (reinterpret_cast<uintptr_t>(x) & 15)) return false;
  if (T > 0x7fffffffLL || C / 32 > 0x7fffffffLL) return false;
  return encode_tiled_fn() != nullptr;
}

cudaError_t fb4_launch_quantize_fast_f32(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld,
                                         uint8_t* codes, uint16_t* meta, cudaStream_t stream) {
  CUtensorMap map;
  const cuuint64_t dims[3] = {32, (cuuint64_t)(C / 32), (cuuint64_t)T};
  const cuuint64_t strides[2] = {128, (cuuint64_t)ld * 4};
  const cuuint32_t box[3] = {32, 32, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const cudaError_t ce = cached_tensor_map(ctx, 3, x, T, C, ld, &map, [&](CUtensorMap* m) {
    return encode_tiled_fn()(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(x), dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  });
  if (ce != cudaSuccess) return ce;
  FastParams p{};
  p.T = T;
  p.C = C;
  p.tiles_per_row = (C + 1023) / 1024;
  p.n_tiles = T * p.tiles_per_row;
  p.codes = codes;
  p.meta = meta;
  p.status = ctx->d_status;
  const int64_t want = (p.n_tiles + kWarpsF32 - 1) / kWarpsF32;
  const int grid = (int)(want < ctx->sm_count ? want : ctx->sm_count);
  const int64_t wstride = (int64_t)grid * kWarpsF32;
  p.step_rows = wstride / p.tiles_per_row;
  p.step_cols = (int32_t)(wstride % p.tiles_per_row);
  fb4_quantize_f32_kernel<<<grid, kWarpsF32 * 32, kSmemBytesF32, stream>>>(
      map, static_cast<const SmemTables*>(ctx->d_fast_tables), p);
  return cudaGetLastError();
}

// Quantize straight to an MXFP8 operand (e4m3 bytes + E8M0 scales): default configuration only.
bool fb4_fast_mx_eligible(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld) {
  const fb4_config& c = ctx->cfg;
  return c.block_size == 32 && c.num_groups == 8 && c.select_mode == 0 && c.exp_min == -124 && c.exp_max == 127 &&
         fb4_fast_eligible(ctx, x, T, C, ld);
}

// With ex.n_salient > 0 the residual of the salient rows goes to res_e4m3 [n_salient][C] and
// res_scales (the scale layout applied to the [n_salient][C] operand); ex.res_codes / res_meta are
// not used.
cudaError_t fb4_launch_quantize_fast_mx(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld,
                                        const Fb4RowExtras& ex, uint8_t* e4m3, uint8_t* scales, uint8_t* res_e4m3,
                                        uint8_t* res_scales, int tiled, cudaStream_t stream, int* launches) {
  const bool decomp = ex.n_salient > 0;
  CUtensorMap map;
  if (flat_eligible(T, C, ld)) {
    FlatParams fp;
    int fgrid = 0;
    cudaError_t fe = flat_setup(ctx, x, T, C, decomp, true, &map, &fp, &fgrid);
    if (fe != cudaSuccess) return fe;
    fp.e4m3 = e4m3;
    fp.scales = scales;
    fp.res_e4m3 = res_e4m3;
    fp.res_scales = res_scales;
    fp.scale_tiled = tiled;
    const int64_t n_col = C / 32;
    fp.scale_col_tiles = (n_col + 3) / 4;
    // the kernel writes real entries only: padding of the tiled layout = scale 1
    if (tiled && ((T & 127) || (n_col & 3))) {
      fe = cudaMemsetAsync(scales, 0x7f, (size_t)(((T + 127) / 128) * fp.scale_col_tiles * 512), stream);
      if (fe != cudaSuccess) return fe;
    }
    if (decomp && tiled && ((ex.n_salient & 127) || (n_col & 3))) {
      fe = cudaMemsetAsync(res_scales, 0x7f, (size_t)(((ex.n_salient + 127) / 128) * fp.scale_col_tiles * 512), stream);
      if (fe != cudaSuccess) return fe;
    }
    const SmemTables* ftables = static_cast<const SmemTables*>(ctx->d_fast_tables);
#define FB4_MXF(S, D) \
  fb4_quantize_flat_kernel<S, D, false, false, true><<<fgrid, kWarps * 32, kSmemBytes, stream>>>(map, ftables, fp, ex)
    switch ((ex.cluster_id ? 1 : 0) | (decomp ? 2 : 0)) {
      case 0: FB4_MXF(false, false); break;
      case 1: FB4_MXF(true, false); break;
      case 2: FB4_MXF(false, true); break;
      default: FB4_MXF(true, true); break;
    }
#undef FB4_MXF
    fe = cudaGetLastError();
    if (fe == cudaSuccess) *launches = 1;
    return fe;
  }
  FastParams p;
  int grid = 0;
  cudaError_t e = fast_setup(ctx, x, T, C, ld, decomp, &map, &p, &grid);
  if (e != cudaSuccess) return e;
  p.e4m3 = e4m3;
  p.scales = scales;
  p.res_e4m3 = res_e4m3;
  p.res_scales = res_scales;
  p.scale_tiled = tiled;
  const int64_t n_col = C / 32;
  p.scale_col_tiles = (n_col + 3) / 4;
  // the kernel writes real entries only: padding of the tiled layout = scale 1
  if (tiled && ((T & 127) || (n_col & 3))) {
    e = cudaMemsetAsync(scales, 0x7f, (size_t)(((T + 127) / 128) * p.scale_col_tiles * 512), stream);
    if (e != cudaSuccess) return e;
  }
  if (decomp && tiled && ((ex.n_salient & 127) || (n_col & 3))) {
    e = cudaMemsetAsync(res_scales, 0x7f, (size_t)(((ex.n_salient + 127) / 128) * p.scale_col_tiles * 512), stream);
    if (e != cudaSuccess) return e;
  }
  const SmemTables* tables = static_cast<const SmemTables*>(ctx->d_fast_tables);
  const int variant = (ex.cluster_id ? 1 : 0) | (decomp ? 2 : 0);
#define FB4_MX(S, D) \
  fb4_quantize_fast_kernel<S, D, false, false, true><<<grid, kWarps * 32, kSmemBytes, stream>>>(map, tables, p, ex)
  switch (variant) {
    case 0: FB4_MX(false, false); break;
    case 1: FB4_MX(true, false); break;
    case 2: FB4_MX(false, true); break;
    default: FB4_MX(true, true); break;
  }
#undef FB4_MX
  e = cudaGetLastError();
  if (e == cudaSuccess) *launches = 1;
  return e;
}

// The same helpers for the kernels of fb4_producers.cu.
cudaError_t fb4_fast_setup(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, bool chunked,
                           CUtensorMap* map, fb4stage::FastParams* p, int* grid_out) {
  return fast_setup(ctx, x, T, C, ld, chunked, map, p, grid_out);
}
cudaError_t fb4_flat_setup(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, bool chunked, bool mx,
                           CUtensorMap* map, fb4stage::FlatParams* p, int* grid_out) {
  return flat_setup(ctx, x, T, C, chunked, mx, map, p, grid_out);
}
bool fb4_flat_eligible(int64_t T, int64_t C, int64_t ld) { return flat_eligible(T, C, ld); }
