// Token-column tiles of the row-space grouped GEMMs (GMM1+SwiGLU, GMM2, act_grad, gate_grad) on CTA
// pairs.  The weights take the 256 accumulator ROWS of a pair (128 per CTA, the A operand of
// tcgen05.mma) and the expert's tokens the accumulator COLUMNS (the B operand, 32..256 per tile in
// steps of 32, half of them in each CTA's shared memory).  The MMA time of a tile then follows the
// number of tokens it really holds instead of the padded 256 rows of a token-row tile.
//
// The accumulator arrives transposed (TMEM lane = output feature, column = token); the epilogues
// write it back token-major through small un-swizzled staging boxes and TMA stores.
#pragma once

#include <cuda_bf16.h>

#include "gemm_pair.cuh"

namespace moe {

constexpr int TOK_GRAIN = 32;                    // tokens per tile: a multiple of 32 (16 rows of B per CTA)
constexpr int W_STAGE_BYTES = A_STAGE_BYTES;     // 128 weight rows (or 2 MN-major boxes) x 64 k: 16 KB
constexpr int SW_SLOT_BYTES = 4096;              // one staging slot of an epilogue warp
#ifndef MOE_SW_SLOTS
#define MOE_SW_SLOTS 2
#endif
constexpr int SW_SLOTS = MOE_SW_SLOTS;           // ring of slots per warp

struct SwapTile {
  int e;      // expert
  int row0;   // first padded row of the tile's tokens
  int ntok;   // tokens (accumulator columns) of the tile, multiple of TOK_GRAIN
  int n0;     // first output feature of the pair (GATE_UP: of the 128 gate/up feature pairs)
  int nb;     // feature-tile index
  int nkb;    // k-blocks
  int mb_first, mb_count;   // the tile's M-blocks (its event counters)
};

// Features per pair tile: GATE_UP holds 64 gate + 64 up rows per CTA = 128 features per pair.
template <int MODE>
__device__ __forceinline__ int swap_tile_features() { return MODE == GEMM_GATE_UP ? 128 : 256; }

// Tokens of the unit of M-blocks [first, first + count) (relative to the expert's first M-block) of expert e,
// cut at the expert's last 32-row group.
__device__ __forceinline__ void unit_tokens(const GemmArgs& a, int e, int first, int count, int* row0, int* ntok) {
  const int n32 = (a.counts[e] + TOK_GRAIN - 1) & ~(TOK_GRAIN - 1);
  int end = (first + count) * BLOCK_M;
  if (end > n32) end = n32;
  *row0 = (a.mb_start[e] + first) * BLOCK_M;
  *ntok = end - first * BLOCK_M;
}

// One work item of a row-space operator: a token tile, or -- in the operators that merge,
// for an expert with an odd count of three or more M-blocks -- its last two token tiles (one block;
// block + tail) under ONE k-loop: the weight stage is written to shared memory once and multiplied with
// both token tiles into the two TMEM accumulators (shared-memory traffic bounds these kernels, and the
// weights are the larger half of it).  For the epilogue warps the item is two consecutive tiles.
// Only the operators with a short epilogue merge (down, gate_grad): with both accumulators in use the
// epilogue of the second tile is exposed.
struct SwapWork {
  SwapTile a, b;
  bool merged;
};
template <int MODE>
__host__ __device__ constexpr bool swap_merges() { return MODE == GEMM_DOWN || MODE == GEMM_GATE_GRAD; }
// token bytes of a stage per CTA: up to 128 rows, or (128 + 256) / 2 rows of a merged item
template <int MODE>
__host__ __device__ constexpr int tok_stage_bytes() { return (swap_merges<MODE>() ? 3 : 2) * 64 * BK * 2; }

template <int MODE>
__device__ __forceinline__ int total_swap_work(const GemmArgs& a) {
  return (swap_merges<MODE>() ? a.meta[4] : a.meta[3]) * a.n_tiles_n;
}

// Item order: expert-major; inside an expert the feature tile is the slow index and the item the
// fast one (items running at the same time share one slab of weights in L2).
template <int MODE>
__device__ __forceinline__ SwapWork decode_swap_work(const GemmArgs& a, int t) {
  constexpr bool mg = swap_merges<MODE>();
  const SwapItem it = decode_swap_item(t, a.n_tiles_n, mg, mg ? a.work_start : a.pair_start,
                                       mg ? a.wblk_expert : a.pblk_expert, a.mb_start);
  SwapWork w;
  w.merged = it.merged != 0;
  w.a.e = w.b.e = it.e;
  w.a.nb = w.b.nb = it.nb;
  w.a.n0 = w.b.n0 = it.nb * swap_tile_features<MODE>();
  w.a.nkb = w.b.nkb = (a.K + BK - 1) / BK;
  const int rel = it.mb_first - a.mb_start[it.e];
  unit_tokens(a, it.e, rel, it.mb_count_a, &w.a.row0, &w.a.ntok);
  w.a.mb_first = it.mb_first; w.a.mb_count = it.mb_count_a;
  w.b.row0 = 0; w.b.ntok = 0;
  w.b.mb_first = it.mb_first + it.mb_count_a; w.b.mb_count = it.mb_count - it.mb_count_a;
  if (w.merged) unit_tokens(a, it.e, rel + it.mb_count_a, w.b.mb_count, &w.b.row0, &w.b.ntok);
  return w;
}

__device__ __forceinline__ uint32_t swap_stage_tx_bytes(int ntok) {
  return 2u * (uint32_t)(W_STAGE_BYTES + (ntok >> 1) * BK * 2);   // both CTAs: weights + half of the tokens
}

// This CTA's loads of one k-block are split over two producer warps, one box per lane (issuing a TMA
// box costs its thread on the order of a hundred cycles, and a k-block of a short tile only lasts a
// few hundred).  Tokens: rows [row0 + rank * ntok/2, + ntok/2) as ONE box (a tensor map per box height).  The even CTA's weight producer arms the barrier for both CTAs' bytes.
__device__ __forceinline__ void load_tokens_swap(const GemmArgs& a, const SwapTile& st, int kb, int rank, uint8_t* sT,
                                                 uint64_t* bar, int lane) {
  if (lane != 0) return;
  const int half = st.ntok >> 1;   // a multiple of 16, at most 128: one box of exactly that many rows
  tma_load_2d_pair(sT, &a.tmTok[(half >> 4) - 1], kb * BK, st.row0 + rank * half, bar);
}
template <int MODE>
__device__ __forceinline__ void load_weights_swap(const GemmArgs& a, const SwapTile& st, int kb, int rank, uint8_t* sW,
                                                  uint64_t* bar, int lane, int ntok_total = -1) {
  const int k0 = kb * BK;
  if (lane == 0 && rank == 0) mbar_expect_tx(bar, swap_stage_tx_bytes(ntok_total < 0 ? st.ntok : ntok_total));
  __syncwarp();
  const int brow = st.e * a.b_rows_per_expert;
  if (MODE == GEMM_GATE_UP) {
    // one box [4 groups][gate | up][16 rows][64 k]: per epilogue warp 16 gate rows, then the 16 up rows
    // of the same features (W_gate_up viewed as [Ep][F/16][2][16][d])
    if (lane == 0) tma_load_5d_pair(sW, &a.tmB, k0, 0, 0, (st.n0 + rank * 64) >> 4, st.e, bar);
  } else if (MODE == GEMM_DOWN) {
    if (lane == 0) tma_load_2d_pair(sW, &a.tmB, k0, brow + st.n0 + rank * 128, bar);
  } else {
    // ACT_GRAD / GATE_GRAD: the forward weight read along its rows -> two MN-major [64 k][64 features] boxes
    if (lane < 2) tma_load_2d_pair(sW + lane * MN_BOX_BYTES, &a.tmB, st.n0 + (2 * rank + lane) * 64, brow + k0, bar);
  }
}

// One 64-deep k-block: D[256 features x ntok tokens] (+)= W . X^T.  w_lo / t_lo: low descriptor words of
// the stage's weight and token tiles (smem_desc_lo); the issuing thread only adds the k-step.
template <int MODE>
__device__ __forceinline__ void mma_kblock_swap(uint32_t d_tmem, uint32_t w_lo, uint32_t t_lo, uint32_t idesc,
                                                bool first_kblock) {
  constexpr bool W_MN = (MODE == GEMM_ACT_GRAD || MODE == GEMM_GATE_GRAD);
  constexpr uint32_t hi = smem_desc_hi(1024);
  constexpr uint32_t wstep = W_MN ? (2048 >> 4) : (32 >> 4);   // 16 k-rows of an MN-major box / 32 bytes of a K-major row
#pragma unroll
  for (int k16 = 0; k16 < BK / 16; ++k16)
    tc_mma_bf16_pair_lohi(d_tmem, w_lo + k16 * wstep, hi, t_lo + k16 * 2, hi, idesc, !(first_kblock && k16 == 0));
}
template <int MODE>
__device__ __forceinline__ uint32_t swap_w_desc_lo(uint32_t w_addr) {
  constexpr bool W_MN = (MODE == GEMM_ACT_GRAD || MODE == GEMM_GATE_GRAD);
  return smem_desc_lo(w_addr, W_MN ? MN_BOX_BYTES : 16);
}
template <int MODE>
__device__ __forceinline__ uint32_t swap_idesc(int ntok) {
  constexpr bool W_MN = (MODE == GEMM_ACT_GRAD || MODE == GEMM_GATE_GRAD);
  return make_idesc_bf16(2 * BLOCK_M, ntok, W_MN ? 1 : 0, 0);
}

// ---------------------------------------------------------------- staging ring of an epilogue warp
struct SwStaging {
  uint8_t* base;     // SW_SLOTS slots of SW_SLOT_BYTES
  uint32_t round;
  uint8_t* scratch;  // act_grad: 4 KB of this warp (two halves of [gate | up][16 tokens][32 features])
  uint32_t slots;       // staging slots of this warp (1 or 2)
  uint32_t slot_bytes;  // SW_SLOT_BYTES, or 2 KB in the plain-store operators that give room to the operand stages
};
constexpr int SW_SCRATCH_BYTES = 4096;
__device__ __forceinline__ uint8_t* sw_acquire(SwStaging& sg, int lane) {
  if (lane == 0) {   // the slot's previous stores have read it
    if (sg.slots == 1) tma_store_wait_read();
    else tma_store_wait_read_n<SW_SLOTS - 1>();
  }
  __syncwarp();
  uint8_t* slot = sg.base + (sg.round % sg.slots) * sg.slot_bytes;
  ++sg.round;
  return slot;
}
__device__ __forceinline__ uint16_t bf16_bits(float x) { return __bfloat16_as_ushort(__float2bfloat16_rn(x)); }
__device__ __forceinline__ float bf16_to_f32(uint16_t h) { return __uint_as_float(static_cast<uint32_t>(h) << 16); }
__device__ __forceinline__ uint4 ld_nc_v4(const uint16_t* p) {
  uint4 r;
  asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
  return r;
}


// ---------------------------------------------------------------- epilogues (transposed accumulator)
// Warp `quad` of CTA `rank` owns TMEM lanes 32*quad .. 32*quad+31 (32 output features) and walks the
// tile's tokens 32 columns at a time.  A thread (= one feature) writes one bf16 per token into a
// staging box laid out [token][feature]; lane 0 stores the box with TMA (clipped at the tensor edge).
template <int MODE>
__device__ __forceinline__ void epilogue_swap(const GemmArgs& a, const SwapTile& st, uint32_t tmem_acc, int rank,
                                              int quad, int lane, SwStaging& sg) {
  const uint32_t trow = tmem_acc + (static_cast<uint32_t>(quad * 32) << 16);
  if (MODE == GEMM_DOWN || MODE == GEMM_GATE_GRAD) {
    const int f0 = st.n0 + rank * 128 + quad * 32;   // first output column of this warp
    if (f0 >= a.N) return;
#pragma unroll 1
    for (int c0 = 0; c0 < st.ntok; c0 += 32) {
      float v[32];
      tmem_ld16(trow + c0, v);
      tmem_ld16(trow + c0 + 16, v + 16);
      tmem_ld_wait();
      uint8_t* box = sw_acquire(sg, lane);
      // [32 tokens][32 features].  Neighbouring lanes (features 2i, 2i+1) swap one value per token pair, so that
      // every lane stores 4 bytes: the even lane the feature pair of token j, the odd lane that of token j+1 -- 128
      // contiguous bytes per warp store instead of 64.
      uint32_t* box32 = reinterpret_cast<uint32_t*>(box) + (lane >> 1);
      const bool odd = lane & 1;
#pragma unroll
      for (int j = 0; j < 32; j += 2) {
        const float send = odd ? v[j] : v[j + 1];
        const float recv = __shfl_xor_sync(0xffffffffu, send, 1);
        box32[(j + (odd ? 1 : 0)) * 16] = odd ? pack_bf16x2(recv, v[j + 1]) : pack_bf16x2(v[j], recv);
      }
      staging_release();
      if (lane == 0) {
        tma_store_2d(&a.tmOut0, f0, st.row0 + c0, box);
        tma_store_commit();
      }
    }
  } else if (MODE == GEMM_GATE_UP) {
    // lanes 0..15: gate pre-activations of 16 features, lanes 16..31: up pre-activations of the same
    // features.  For a token pair (j, j+1) the halves swap one value: the low half finishes token j,
    // the high half token j+1.
    const int fl = lane & 15;
    const bool hi = lane >= 16;
    const int fw0 = st.n0 + rank * 64 + quad * 16;   // first feature of this warp
    if (fw0 >= a.F) return;
#pragma unroll 1
    for (int c0 = 0; c0 < st.ntok; c0 += 32) {
      float v[32];
      tmem_ld16(trow + c0, v);
      tmem_ld16(trow + c0 + 16, v + 16);
      const float wl = a.prow_w[st.row0 + c0 + lane];   // routing weight of token c0 + lane
      tmem_ld_wait();
      uint8_t* box = sw_acquire(sg, lane);
      uint16_t* abox = reinterpret_cast<uint16_t*>(box);           // A: [32 tokens][16 features]
      uint16_t* hbox = reinterpret_cast<uint16_t*>(box + 1024 + (hi ? 1024 : 0));   // H gate / H up
#pragma unroll
      for (int j = 0; j < 32; j += 2) {
        const float send = hi ? v[j] : v[j + 1];
        const float recv = __shfl_xor_sync(0xffffffffu, send, 16);
        const float g = hi ? recv : v[j];
        const float u = hi ? v[j + 1] : recv;
        const int tj = j + (hi ? 1 : 0);
        const float w = __shfl_sync(0xffffffffu, wl, tj);
        abox[tj * 16 + fl] = bf16_bits(w * (g * sigmoidf_fast(g) * u));
      }
      if (a.save_h) {
#pragma unroll
        for (int j = 0; j < 32; ++j) hbox[j * 16 + fl] = bf16_bits(v[j]);
      }
      staging_release();
      if (lane == 0) {
        tma_store_2d(&a.tmOut0, fw0, st.row0 + c0, box);
        if (a.save_h) {
          tma_store_3d(&a.tmOut1, fw0, 0, st.row0 + c0, box + 1024);
          tma_store_3d(&a.tmOut1, fw0, 1, st.row0 + c0, box + 2048);
        }
        tma_store_commit();
      }
    }
  } else if (MODE == GEMM_ACT_GRAD) {
    const int f0 = st.n0 + rank * 128 + quad * 32;
    const int nparts = a.n_tiles_n * DW_PARTS_PER_TILE;
    const int slot = (st.nb * 2 + rank) * 4 + quad;
    if (f0 >= a.F) {
      // no features here: the partial slots of this warp still take part in the reduction
      if (a.dw_partial)
        for (int j = lane; j < st.ntok; j += 32) a.dw_partial[(size_t)(st.row0 + j) * nparts + slot] = 0.f;
      return;
    }
    // The saved pre-activations of 16 tokens x 32 features (gate and up: 1 KB each) come in as four
    // 16-byte loads per lane (lane -> token (lane + 32 i) / 4, features 8 (lane % 4) ..), are parked in
    // this warp's scratch [gate | up][16 tokens][32 features] and read back one feature column per lane.
    // The loads of the next 16 tokens are in flight while the current ones are worked on.
    const int part = lane & 3;
    const bool cvalid = f0 + part * 8 < a.F;     // F % 8 == 0: a 16-byte chunk is inside or outside as a whole
    const uint16_t* hbase = a.in0 + (size_t)st.row0 * a.ld_in0 + f0 + part * 8;
    uint4 pre[4];
    auto fetch = [&](int tok0) {
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int t = (lane + 32 * i) >> 2;
        const uint16_t* p = hbase + (size_t)(tok0 + t) * a.ld_in0;
        pre[2 * i] = cvalid ? ld_nc_v4(p) : make_uint4(0, 0, 0, 0);
        pre[2 * i + 1] = cvalid ? ld_nc_v4(p + a.F) : make_uint4(0, 0, 0, 0);
      }
    };
    fetch(0);
    uint8_t* box = nullptr;
    float wl = 0.f;
#pragma unroll 1
    for (int h0 = 0; h0 < st.ntok; h0 += 16) {
      const int hh = h0 & 16;   // which half of the 32-token staging box
      if (hh == 0) {
        box = sw_acquire(sg, lane);
        wl = a.prow_w[st.row0 + h0 + lane];
      }
      uint8_t* scr = sg.scratch + (((h0 >> 4) & 1) ? 2048 : 0);
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int t = (lane + 32 * i) >> 2;
        *reinterpret_cast<uint4*>(scr + t * 64 + part * 16) = pre[2 * i];
        *reinterpret_cast<uint4*>(scr + 1024 + t * 64 + part * 16) = pre[2 * i + 1];
      }
      if (h0 + 16 < st.ntok) fetch(h0 + 16);
      float da[16], pr[16];
      tmem_ld16(trow + h0, da);
      __syncwarp();
      tmem_ld_wait();
      uint16_t* gbox = reinterpret_cast<uint16_t*>(box) + lane;          // d(gate): [32 tokens][32 features]
      uint16_t* ubox = reinterpret_cast<uint16_t*>(box + 2048) + lane;   // d(up)
      const uint16_t* gs16 = reinterpret_cast<const uint16_t*>(scr) + lane;
      const uint16_t* us16 = reinterpret_cast<const uint16_t*>(scr + 1024) + lane;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float g = bf16_to_f32(gs16[j * 32]), u = bf16_to_f32(us16[j * 32]);
        const float s = sigmoidf_fast(g);
        const float gs = g * s;
        pr[j] = da[j] * (gs * u);                   // <dA_unweighted, a>: gradient of the routing weight
        const float w = __shfl_sync(0xffffffffu, wl, hh + j);
        const float dav = w * da[j];                // backward Dispatch's weight, applied here
        gbox[(hh + j) * 32] = bf16_bits(dav * u * (s * (1.0f + g * (1.0f - s))));
        ubox[(hh + j) * 32] = bf16_bits(dav * gs);
      }
      if (a.dw_partial) {
        // sum over the warp's 32 features: a transposing butterfly leaves token (lane >> 1) in each lane
#pragma unroll
        for (int off = 16, n = 8; off >= 2; off >>= 1, n >>= 1) {
          const bool up = (lane & off) != 0;
#pragma unroll
          for (int i = 0; i < n; ++i) {
            const float keep = up ? pr[i + n] : pr[i];
            const float send = up ? pr[i] : pr[i + n];
            pr[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
          }
        }
        pr[0] += __shfl_xor_sync(0xffffffffu, pr[0], 1);
        if ((lane & 1) == 0) a.dw_partial[(size_t)(st.row0 + h0 + (lane >> 1)) * nparts + slot] = pr[0];
      }
      if (hh == 16) {
        staging_release();
        if (lane == 0) {
          tma_store_3d(&a.tmOut0, f0, 0, st.row0 + h0 - 16, box);
          tma_store_3d(&a.tmOut0, f0, 1, st.row0 + h0 - 16, box + 2048);
          tma_store_commit();
        }
      } else {
        __syncwarp();   // the scratch half written two rounds from now is the one just read
      }
    }
  }
}

}  // namespace moe
