// Tile-level building blocks of the grouped GEMMs on the sm_100a tensor cores: tile geometry and the
// fused epilogues of the token-row tiles (TMEM -> registers -> element-wise math -> swizzled shared
// staging -> TMA store).
//
// Tiles never straddle experts: rows live in a padded row space where every expert segment starts
// on a multiple of 128 (the paper's rule that vector tiles align with GMM row partitions and that
// the reduction dimension stays intact, Section 4.2).
#pragma once

#include "moe_internal.h"

namespace moe {


constexpr int BN = 256;                       // accumulator columns per tile
constexpr int BK = 64;                        // reduction elements per stage (one 128-byte swizzle row)
constexpr int A_STAGE_BYTES = BLOCK_M * BK * 2;  // 16 KB
constexpr int B_STAGE_BYTES = BN * BK * 2;       // 32 KB
constexpr int MN_BOX_BYTES = 64 * BK * 2;        // one [64 k][64 mn] box of an MN-major operand
constexpr int GEMM_THREADS = 192;
constexpr int TMEM_COLS = 512;
constexpr int OUT_BOX_BYTES = 32 * 64 * 2;       // epilogue staging box: 32 rows x 64 bf16 columns
constexpr int OUT_STAGE_BYTES = 2 * OUT_BOX_BYTES;  // per epilogue warp: two boxes

struct Tile {
  int e;      // expert
  int row0;   // row-space modes: first padded row of the M-block; WGRAD: first padded row of the expert
  int n0;     // first output column of the tile
  int m0;     // WGRAD: first output row (within the expert's slab)
  int nkb;    // k-blocks of the main loop (may be 0 for an expert without rows in WGRAD)
  int nb;     // column-tile index (ACT_GRAD partials)
};

// ---------------------------------------------------------------- epilogues
// Each epilogue warp owns 32 rows of the tile (its TMEM lane quadrant) and a private staging area of
// two [32 rows][64 columns] bf16 boxes in the 128-byte-swizzled layout the store tensor maps expect.
// A thread (= one row) writes 16-byte chunks at chunk index (j ^ (row & 7)): conflict-free.
__device__ __forceinline__ void stage8(uint8_t* box, int lane, int j, const float* v) {
  uint4 q = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]),
                       pack_bf16x2(v[6], v[7]));
  *reinterpret_cast<uint4*>(box + lane * 128 + ((j ^ (lane & 7)) << 4)) = q;
}
__device__ __forceinline__ void load8_bf16(const uint16_t* p, float* v) {
  uint4 r;
  asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
  v[0] = bf16lo(r.x); v[1] = bf16hi(r.x); v[2] = bf16lo(r.y); v[3] = bf16hi(r.y);
  v[4] = bf16lo(r.z); v[5] = bf16hi(r.z); v[6] = bf16lo(r.w); v[7] = bf16hi(r.w);
}
__device__ __forceinline__ float sigmoidf_fast(float g) { return __fdividef(1.0f, 1.0f + __expf(-g)); }

// Before refilling the staging area: the previous stores must have finished reading it.
// `nbuf` staging areas are used round-robin: with two, the stores of one round drain while the next
// round is being filled.
struct Staging {
  uint8_t* base;
  uint32_t nbuf;   // 1 or 2 areas of OUT_STAGE_BYTES
  uint32_t round;
};
__device__ __forceinline__ uint8_t* staging_acquire(Staging& sg, int lane) {
  if (lane == 0) {
    if (sg.nbuf == 2) tma_store_wait_read1();
    else tma_store_wait_read();
  }
  __syncwarp();
  uint8_t* area = sg.base + (sg.round % sg.nbuf) * OUT_STAGE_BYTES;
  ++sg.round;
  return area;
}
// After filling: publish the writes to the async proxy; lane 0 then issues the stores.
__device__ __forceinline__ void staging_release() {
  fence_proxy_async_smem();
  __syncwarp();
}

template <int MODE>
__device__ __forceinline__ void epilogue_tile(const GemmArgs& a, const Tile& tl, uint32_t tmem_acc, int quad,
                                              int lane, Staging& sg) {
  const uint32_t trow = tmem_acc + (static_cast<uint32_t>(quad * 32) << 16);
  uint8_t *box0, *box1;
  if (MODE == GEMM_GATE_UP) {
    const int prow0 = tl.row0 + quad * 32;             // first padded row of this warp's slab
    const float w = a.prow_w[prow0 + lane];
    // first pass over the accumulator: A = w * silu(g) * u, 128 columns
    box0 = staging_acquire(sg, lane); box1 = box0 + OUT_BOX_BYTES;
    for (int c = 0; c < BN / 2; c += 16) {
      float g[16], u[16], act[16];
      tmem_ld16(trow + c, g);
      tmem_ld16(trow + BN / 2 + c, u);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 16; ++i) act[i] = w * (g[i] * sigmoidf_fast(g[i]) * u[i]);
      uint8_t* box = (c < 64) ? box0 : box1;
      stage8(box, lane, (c & 63) >> 3, act);
      stage8(box, lane, ((c & 63) >> 3) + 1, act + 8);
    }
    staging_release();
    if (lane == 0) {
      tma_store_2d(&a.tmOut0, tl.n0, prow0, box0);
      if (tl.n0 + 64 < a.F) tma_store_2d(&a.tmOut0, tl.n0 + 64, prow0, box1);
      tma_store_commit();
    }
    if (a.save_h) {
      // second and third pass: the pre-activations, kept for the backward pass (H viewed as [row][gate|up][F])
#pragma unroll 1
      for (int half = 0; half < 2; ++half) {
        box0 = staging_acquire(sg, lane); box1 = box0 + OUT_BOX_BYTES;
        for (int c = 0; c < BN / 2; c += 16) {
          float v[16];
          tmem_ld16(trow + half * (BN / 2) + c, v);
          tmem_ld_wait();
          uint8_t* box = (c < 64) ? box0 : box1;
          stage8(box, lane, (c & 63) >> 3, v);
          stage8(box, lane, ((c & 63) >> 3) + 1, v + 8);
        }
        staging_release();
        if (lane == 0) {
          tma_store_3d(&a.tmOut1, tl.n0, half, prow0, box0);
          if (tl.n0 + 64 < a.F) tma_store_3d(&a.tmOut1, tl.n0 + 64, half, prow0, box1);
          tma_store_commit();
        }
      }
    }
  } else if (MODE == GEMM_ACT_GRAD) {
    const int prow0 = tl.row0 + quad * 32;
    const size_t p = (size_t)prow0 + lane;
    const float w = a.prow_w[p];
    const uint16_t* hrow = a.in0 + p * a.ld_in0;
    float part = 0.f;
    // 64 columns of F per round: box0 <- d(gate), box1 <- d(up)
#pragma unroll 1
    for (int c0 = 0; c0 < BN; c0 += 64) {
      if (tl.n0 + c0 >= a.F) break;  // uniform: whole round outside the tensor
      box0 = staging_acquire(sg, lane); box1 = box0 + OUT_BOX_BYTES;
#pragma unroll
      for (int c = 0; c < 64; c += 16) {
        float da[16];
        tmem_ld16(trow + c0 + c, da);
        tmem_ld_wait();
#pragma unroll
        for (int h = 0; h < 16; h += 8) {
          const int col = tl.n0 + c0 + c + h;
          float g[8], u[8], dg[8], du[8];
          if (col < a.F) {
            load8_bf16(hrow + col, g);
            load8_bf16(hrow + a.F + col, u);
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) g[i] = u[i] = 0.f;
          }
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float s = sigmoidf_fast(g[i]);
            const float gs = g[i] * s;
            part += da[h + i] * (gs * u[i]);        // <dA_unweighted, a>: gradient of the routing weight
            const float dav = w * da[h + i];        // backward Dispatch's weight, applied here
            dg[i] = dav * u[i] * (s * (1.0f + g[i] * (1.0f - s)));
            du[i] = dav * gs;
          }
          stage8(box0, lane, (c + h) >> 3, dg);
          stage8(box1, lane, (c + h) >> 3, du);
        }
      }
      staging_release();
      if (lane == 0) {
        tma_store_3d(&a.tmOut0, tl.n0 + c0, 0, prow0, box0);
        tma_store_3d(&a.tmOut0, tl.n0 + c0, 1, prow0, box1);
        tma_store_commit();
      }
    }
    if (a.dw_partial) a.dw_partial[p * a.n_tiles_n + tl.nb] = part;
  } else {
    // plain bf16 store of the accumulator: DOWN (Y), GATE_GRAD (dXp)
    const int y0 = tl.row0 + quad * 32;
#pragma unroll 1
    for (int c0 = 0; c0 < BN; c0 += 128) {
      if (tl.n0 + c0 >= a.N) break;
      box0 = staging_acquire(sg, lane); box1 = box0 + OUT_BOX_BYTES;
#pragma unroll
      for (int c = 0; c < 128; c += 64) {
        // 64 columns per TMEM round trip (one wait per box)
        float v[64];
#pragma unroll
        for (int q = 0; q < 4; ++q) tmem_ld16(trow + c0 + c + 16 * q, v + 16 * q);
        tmem_ld_wait();
        uint8_t* box = (c < 64) ? box0 : box1;
#pragma unroll
        for (int h = 0; h < 64; h += 8) stage8(box, lane, h >> 3, v + h);
      }
      staging_release();
      if (lane == 0) {
        tma_store_2d(&a.tmOut0, tl.n0 + c0, y0, box0);
        if (tl.n0 + c0 + 64 < a.N) tma_store_2d(&a.tmOut0, tl.n0 + c0 + 64, y0, box1);
        tma_store_commit();
      }
    }
  }
}

}  // namespace moe
