// What the TMA-staged kernels share: the per-warp ring (constants, mbarrier / TMA / bulk-copy wrappers with
// bounded waits left to the caller), the launch parameter blocks of the strided and the flat tile walks, and the
// host helpers that encode a tensor map and fill those blocks.  Included by fb4_fast.cu (the quantize kernels)
// and fb4_producers.cu (the kernels with a producer fused in front).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "fb4_block.cuh"
#include "fb4_internal.h"

namespace fb4stage {

using SmemTables = fb4blk::Tables;

constexpr int kWarps = 16;           // warps per CTA
constexpr int kStages = 4;           // ring depth per warp
constexpr int kTileBytes = 2048;     // 1024 bf16
constexpr uint32_t kSpinLimit = 1u << 20;   // tries per wait before a warp gives up

struct FastParams {
  int64_t T, C;
  int64_t tiles_per_row, n_tiles;
  int64_t step_rows;    // gridDim.x*kWarps tiles ahead = step_rows rows + step_cols tile columns
  int32_t step_cols;
  uint8_t* codes;
  uint16_t* meta;
  uint32_t* status;   // device word: bit 0 = a TMA wait ran out
  uint32_t ec_lo, ec_hi;   // clamp of the biased block exponent (CLAMP kernels): exp_min + 127, exp_max + 127
  uint8_t* e4m3;           // MX kernels: e4m3 bytes [T][C] and E8M0 scale bytes instead of codes / meta
  uint8_t* scales;
  uint8_t* res_e4m3;       // MX kernels with residual pass: the residual rows in the same form
  uint8_t* res_scales;
  int64_t scale_col_tiles;
  int32_t scale_tiled;
};

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ void tma_load_tile(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c_outer,
                                              int row) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(0), "r"(c_outer), "r"(row) : "memory");
}
// untiled bulk copy global -> shared, completing on an mbarrier (addresses and size multiples of 16)
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

struct FlatParams {
  uint32_t n_tiles;        // tiles; the last one may reach beyond the tensor (TMA fills zeros, stores are guarded)
  uint32_t n_units;        // 32-element units in the tensor (even)
  uint32_t units_row;      // units per token (even)
  uint32_t step_rows;      // one warp step (units between a warp's consecutive tiles) = step_rows tokens + step_rem units
  uint32_t step_rem;
  uint8_t* codes;
  uint16_t* meta;
  uint32_t* status;
  uint32_t ec_lo, ec_hi;
  uint8_t* e4m3;           // MX: e4m3 bytes and E8M0 scale bytes instead of codes / meta
  uint8_t* scales;
  uint8_t* res_e4m3;
  uint8_t* res_scales;
  int64_t scale_col_tiles;
  int32_t scale_tiled;
};

struct FlatPos {
  int32_t row;      // token
  uint32_t rem;     // unit inside the token
  __device__ __forceinline__ void advance(const FlatParams& p) {
    row += (int32_t)p.step_rows;
    rem += p.step_rem;
    if (rem >= p.units_row) { rem -= p.units_row; ++row; }
  }
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
// A load that stays where it is written (the compiler may not sink it towards its use): the per-token
// inputs of the tiles ahead are requested before the wait on the current tile.
__device__ __forceinline__ uint32_t ldg_early(const void* ptr) {
  uint32_t v;
  asm volatile("ld.global.nc.b32 %0, [%1];" : "=r"(v) : "l"(ptr));
  return v;
}
__device__ __forceinline__ void stg_v8(void* ptr, const uint32_t* o) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(ptr), "r"(o[0]), "r"(o[1]), "r"(o[2]),
               "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
}

// dynamic shared memory of a 16-warp kernel: alignment slack, ring, table image, ring barriers + table barrier
constexpr size_t kSmemBytes =
    1024 + (size_t)kWarps * kStages * kTileBytes + sizeof(SmemTables) + (kWarps * kStages + 1) * 8;
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget of one CTA");
static_assert(sizeof(SmemTables) % 16 == 0, "bulk copy size; mbarriers behind the tables stay 8-byte aligned");

}  // namespace fb4stage

// Host helpers (fb4_fast.cu).  Tensor map, grid and tile-walk parameters of one launch on the strided view
// [T][C/64][64]; the same for the flat 2-D view [N/64][64] of a contiguous tensor (chunked or mx: one unit per
// lane, 2 KB tiles; else two units, 4 KB tiles); whether a tensor can take the flat view at all.
cudaError_t fb4_fast_setup(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, int64_t ld, bool chunked,
                           CUtensorMap* map, fb4stage::FastParams* p, int* grid_out);
cudaError_t fb4_flat_setup(const fb4_ctx* ctx, const void* x, int64_t T, int64_t C, bool chunked, bool mx,
                           CUtensorMap* map, fb4stage::FlatParams* p, int* grid_out);
bool fb4_flat_eligible(int64_t T, int64_t C, int64_t ld);
// Opt-in to the dynamic shared memory of the producer kernels on the current device (fb4_producers.cu).
cudaError_t fb4_producers_prepare_device();
