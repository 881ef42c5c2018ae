// Host-side declarations shared by the translation units of libmoe_b200: problem dimensions,
// workspace views and the launch functions of each kernel family.
#pragma once

#include <cuda.h>
#include <atomic>
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"
#include "schedule.h"

namespace moe {

struct Dims {
  int T, d, E, k, S, F;
  int Ep() const { return E + S; }
  int kp() const { return k + S; }
  int slots() const { return T * (k + S); }
};

// Row capacity of the padded expert-ordered row space: every expert segment starts on a
// multiple of BLOCK_M, so at most BLOCK_M-1 padding rows per expert.
inline int padded_rows_max(int T_max, int kp, int Ep) {
  long r = (long)T_max * kp + (long)Ep * (BLOCK_M - 1);
  return (int)(((r + BLOCK_M - 1) / BLOCK_M) * BLOCK_M);
}

constexpr int LAYOUT_CHUNK = 2048;  // flat slots per block of the layout kernels (8 warps x 256)

// Device arrays describing one dispatch layout.
struct LayoutView {
  int* counts;       // [Ep]
  int* offsets;      // [Ep+1]  exclusive scan of counts (unpadded rows)
  int* row_of;       // [slots] unpadded row of each slot, -1 if the slot's expert id is invalid
  int* src_of;       // [slots] slot of each unpadded row
  int* prow_of;      // [slots] padded row of each slot (-1 if invalid)
  int* pad_off;      // [Ep+1]  first padded row of each expert (multiple of BLOCK_M)
  int* mb_start;     // [Ep+1]  first M-block of each expert
  int* mblk_expert;  // [R_pad_max / BLOCK_M] expert of each M-block
  int* pair_start;   // [Ep+1]  first M-block pair of each expert (pairs = ceil(M-blocks / 2))
  int* pblk_expert;  // [pairs] expert of each M-block pair
  int* work_start;   // [Ep+1]  first work item of each expert (token-column GEMMs that merge: its units, the last
                     //         two of an odd M-block count >= 3 merged into one item)
  int* wblk_expert;  // [items] expert of each work item
  int* meta;         // [8]     {num_mblocks, R_pad, rows, num_pairs, num_work_items, 0...}
  int* blk_hist;     // [nblk][Ep] per-block histograms, then per-block exclusive prefixes
  int* combine_order; // [T] persistent launch: tokens in the order in which their last row is produced (NULL: token order)
  int* tok_last;      // [T] 1 + largest padded row of each token (0: none); NULL when the combine order is not wanted
};

// ---- route_layout.cu
// gate_mode: bit 0 = renormalise the k scores, bit 1 = sigmoid scores instead of softmax (GATE_RENORM, GATE_SIGMOID)
constexpr int GATE_RENORM = 1, GATE_SIGMOID = 2;
cudaError_t launch_route(const float* logits, int T, int E, int k, int gate_mode, int* topk_ids, float* topk_w,
                         int* counts, cudaStream_t s, int* launches);
cudaError_t launch_layout(const int* topk_ids, const Dims& dm, const LayoutView& lv, DevStatus* status,
                          cudaStream_t s, int* launches);
// process-wide switch of moe_sched_study's persistent launches (diagnostic; see moe_debug_set_plain_launch)
std::atomic<bool>& study_plain_launch();
cudaError_t launch_layout_order(const Dims& dm, const LayoutView& lv, int cap_mblocks, cudaStream_t s, int* launches);

// ---- permute.cu
// Xp[p] = src[token of padded row p] (zeros on padding rows); optionally prow_w[p] = routing weight
// of the row (1 for shared experts, 0 on padding rows).
cudaError_t launch_gather(const uint16_t* src, const float* topk_w, const Dims& dm, const LayoutView& lv,
                          uint16_t* dst, float* prow_w, int rows_cap, cudaStream_t s, int* launches,
                          DevStatus* status = nullptr, uint64_t budget_ns = 0);
// out[t] = sum_j rows[prow_of[t*kp+j]] in slot order, fp32 accumulate, bf16 result; tokens [t0, t1)
// (t1 < 0: all).
cudaError_t launch_combine(const uint16_t* rows, const Dims& dm, const LayoutView& lv, uint16_t* out,
                           cudaStream_t s, int* launches, int t0 = 0, int t1 = -1);
// d_topk_w[t][j] = sum_nb partial[prow_of[t*kp+j]][nb]
cudaError_t launch_dw_reduce(const float* partial, int nparts, const Dims& dm, const LayoutView& lv,
                             float* d_topk_w, cudaStream_t s, int* launches);

// ---- grouped GEMMs (tcgen05 on CTA pairs)
enum GemmMode : int {
  GEMM_GATE_UP = 0,    // H = Xp . W_gate_up[e]^T, epilogue A = w * silu(g) * u     (fwd GMM1 + SwiGLU)
  GEMM_DOWN = 1,       // Y = A . W_down[e]^T                                        (fwd GMM2)
  GEMM_ACT_GRAD = 2,   // dA = dOutp . W_down[e], epilogue SwiGLU_grad -> dH, d_w    (bwd act_grad + SwiGLU_grad)
  GEMM_GATE_GRAD = 3,  // dXp = dH . W_gate_up[e]                                    (bwd gate_grad)
  GEMM_WGRAD = 4,      // dW[e] = P_e^T . Q_e over the expert's rows                 (bwd w1_grad / w2_grad)
};

struct GemmArgs {
  CUtensorMap tmA;     // A operand
  CUtensorMap tmB;     // B operand
  CUtensorMap tmOut0;  // store map of out0: [rows][N] (2-D), [rows][2][F] (dH), or [Ep][M][N] (WGRAD)
  CUtensorMap tmOut1;  // GATE_UP: store map of H as [rows][2][F]
  CUtensorMap tmTok[8]; // token-column tiles: the token operand with boxes of 16, 32, .., 128 rows (one TMA instruction
                        // per k-block whatever the tile's token count)
  // tile table
  const int* mblk_expert;
  const int* mb_start;
  const int* counts;
  const int* meta;
  const int* pair_start;   // CTA-pair kernels: first M-block pair of each expert
  const int* pblk_expert;  // CTA-pair kernels: expert of each M-block pair
  const int* work_start;   // token-column kernel: first work item of each expert
  const int* wblk_expert;  // token-column kernel: expert of each work item
  int cap_rows;            // rows of the padded row space (a row coordinate >= cap_rows reads zeros)
  int Ep;
  int n_tiles_n;       // tiles along N per M-block (row-space modes) / per expert (WGRAD)
  int n_tiles_m;       // WGRAD only: tiles along M per expert
  int K;               // reduction length (row-space modes)
  int N;               // output columns (for masking); WGRAD: columns of dW
  int M;               // WGRAD: rows of dW per expert
  int b_rows_per_expert;  // rows of the B tensor map per expert slab
  int F;               // intermediate size (GATE_UP / ACT_GRAD epilogues)
  // epilogue tensors
  int save_h;          // GATE_UP: also store the pre-activations H
  const uint16_t* in0; // ACT_GRAD: H
  const float* prow_w; // GATE_UP, ACT_GRAD: routing weight per padded row
  float* dw_partial;   // ACT_GRAD: [R_pad][n_tiles_n] partial <dA_unweighted, a> (may be NULL)
  long ld_in0;
  DevStatus* status;
  uint64_t budget_ns;
};

// ---- gemm_tc2.cu: token-row tiles on CTA pairs (tcgen05 cta_group::2, 256 x 256): the row-space operators
// of shapes the token-column tiles do not cover (F % 16 != 0)
cudaError_t launch_gemm2(GemmMode mode, const GemmArgs& a, int num_sms, cudaStream_t s, int* launches);

// ---- gemm_tc3.cu: the row-space operators with the tokens as accumulator COLUMNS (weights take the
// 256 accumulator rows of a CTA pair), so a tile's MMA time follows the expert's real token count
cudaError_t launch_gemm3(GemmMode mode, const GemmArgs& a, int num_sms, cudaStream_t s, int* launches);
// ---- gemm_wgrad.cu: weight gradients strip by strip, the strip's A operand resident in shared memory
cudaError_t launch_wgrad_strips(const GemmArgs& a, int num_sms, cudaStream_t s, int* launches);
constexpr int DW_PARTS_PER_TILE = 8;  // routing-weight gradient partials per (row, column tile): 2 CTAs x 4 warps

// ---- fused.cu (the single persistent dependency-driven launch)
// Everything one fused launch needs: the operators' GEMM arguments (one per phase), the chain
// parameters, the event counters, and the tensors of the vector tasks.
struct FusedArgs {
  GemmArgs op[SCHED_MAX_SEG];
  ChainParams cp;
  LayoutView lv;
  int* ctr;                 // event counters (zeroed before the launch), schedule.h
  int d, kp;
  // gather (Dispatch / backward Dispatch)
  const uint16_t* gather_src;
  uint16_t* gather_dst;
  const float* topk_w;
  float* prow_w;            // written by the forward gather only (may be NULL)
  // combine (Combine / backward Combine)
  const uint16_t* combine_rows;
  uint16_t* combine_out;
  int announce_out;         // 1: count finished combine tasks and set ctr[CTR_OUT_READY] after the last one
  // backward extras
  const float* dw_partial;
  int dw_nparts;
  float* d_topk_w;          // may be NULL
  // per-tile trace (NULL: off)
  uint4* trace;
  int trace_cap;
  DevStatus* status;
  uint64_t budget_ns;
};

// Router in the path (router.cu)
struct RouterArgs {
  CUtensorMap tmX;          // x [T][d] bf16, box 128 rows x 64 columns
  CUtensorMap tmW;          // W_r [E][d] bf16, box N/2 rows x 64 columns (rows beyond E read as zeros)
  int T, E, k, d;
  int N;                    // accumulator columns: E rounded up to a multiple of 16, at least 32, at most 256
  int renorm;               // gate mode bits (GATE_RENORM | GATE_SIGMOID)
  int* topk_ids;
  float* topk_w;
  float* logits;            // may be NULL
  int* counts;              // may be NULL
  DevStatus* status;
  uint64_t budget_ns;
};
cudaError_t launch_router_fwd(const RouterArgs& a, int num_sms, cudaStream_t s, int* launches);
cudaError_t launch_router_bwd(const float* logits, const int* ids, const float* g, int T, int E, int k, int gate_mode,
                              float* dlogits, cudaStream_t s, int* launches);

// cooperative = false drops the co-residency guarantee of the launch (profilers that reject cooperative cluster
// launches); the grid is sized to the resident capacity either way and every wait is bounded
cudaError_t launch_fused(bool bwd, const FusedArgs& fa, int num_sms, bool cooperative, cudaStream_t s, int* launches);

}  // namespace moe
