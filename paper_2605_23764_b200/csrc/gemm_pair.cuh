// Tile-level pieces of the CTA-pair (tcgen05 cta_group::2) grouped GEMMs shared by the
// token-row kernel (gemm_tc2.cu) and the weight gradients (gemm_roles.cuh): each CTA of a pair loads its
// own 128 rows of A and its half of the B tile; the even CTA issues 256 x 256 MMAs.
#pragma once

#include "gemm_tile.cuh"

namespace moe {

constexpr int HALF_B_BYTES = B_STAGE_BYTES / 2;                 // 16 KB: this CTA's half of the B tile
constexpr int STAGE2_BYTES = A_STAGE_BYTES + HALF_B_BYTES;      // 32 KB per stage and CTA

// 16-row MMA steps needed in k-block kb of a reduction over `rows` rows
__device__ __forceinline__ int k16_steps_of(int rows, int kb) {
  const int left = rows - kb * BK;
  return left >= BK ? BK / 16 : (left + 15) / 16;
}

template <int MODE>
__device__ __forceinline__ void mma_kblock_pair(uint32_t d_tmem, uint32_t a_addr, uint32_t b_addr, bool first_kblock,
                                                int k16_steps = BK / 16) {
  constexpr bool A_MN = (MODE == GEMM_WGRAD);
  constexpr bool B_MN = (MODE == GEMM_ACT_GRAD || MODE == GEMM_GATE_GRAD || MODE == GEMM_WGRAD);
  constexpr uint32_t idesc = make_idesc_bf16(2 * BLOCK_M, BN, A_MN ? 1 : 0, B_MN ? 1 : 0);
#pragma unroll
  for (int k16 = 0; k16 < BK / 16; ++k16) {
    const uint64_t da = A_MN ? make_smem_desc(a_addr + k16 * 2048, MN_BOX_BYTES, 1024)
                             : make_smem_desc(a_addr + k16 * 32, 16, 1024);
    const uint64_t db = B_MN ? make_smem_desc(b_addr + k16 * 2048, MN_BOX_BYTES, 1024)
                             : make_smem_desc(b_addr + k16 * 32, 16, 1024);
    // the last k-block of a weight gradient may hold fewer than 64 rows of the expert: the 16-row
    // steps that would only multiply zero padding are not issued
    if (k16 < k16_steps) tc_mma_bf16_pair(d_tmem, da, db, idesc, !(first_kblock && k16 == 0));
  }
}


// The same loads issued by a whole warp, one box per lane.  All lanes call it; in the even CTA lane 0
// arms the barrier for the bytes of both CTAs.
template <int MODE>
__device__ __forceinline__ void load_stage_pair_lanes(const GemmArgs& a, const Tile& tl, int kb, int rank, uint8_t* sA,
                                                      uint8_t* sB, uint64_t* bar, int lane) {
  const int k0 = kb * BK;
  if (lane == 0 && rank == 0) mbar_expect_tx(bar, 2 * STAGE2_BYTES);
  __syncwarp();
  const int brow = tl.e * a.b_rows_per_expert;
  if (lane == 0) {
    tma_load_2d_pair(sA, &a.tmA, k0, tl.row0, bar);
  } else if (MODE == GEMM_GATE_UP) {
    if (lane == 1) tma_load_2d_pair(sB, &a.tmB, k0, brow + rank * a.F + tl.n0, bar);
  } else if (MODE == GEMM_DOWN) {
    if (lane == 1) tma_load_2d_pair(sB, &a.tmB, k0, brow + tl.n0 + rank * (BN / 2), bar);
  } else {
    if (lane < 3)
      tma_load_2d_pair(sB + (lane - 1) * MN_BOX_BYTES, &a.tmB, tl.n0 + (2 * rank + lane - 1) * 64, brow + k0, bar);
  }
}

}  // namespace moe
