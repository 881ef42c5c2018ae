// C ABI of libmoe_b200: context, workspace carving, tensor-map encoding and the launch
// sequences of the forward and backward layer.  Argument marshalling and planning only; every
// step of the layer runs in the kernels of route_layout.cu, permute.cu, gemm_tc3.cu, gemm_wgrad.cu,
// gemm_tc2.cu and fused.cu.
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <string>
#include <vector>

#include "../../include/moe_b200.h"
#include "../../include/moe_b200_debug.h"
#include "moe_internal.h"

using namespace moe;

namespace {

thread_local std::string g_cuda_error;

int cuda_fail(cudaError_t e, const char* what) {
  g_cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
  return MOE_ERR_CUDA;
}
#define MOE_CUDA(call)                                   \
  do {                                                   \
    cudaError_t _e = (call);                             \
    if (_e != cudaSuccess) return cuda_fail(_e, #call);  \
  } while (0)

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Stream memory operations (driver API): a stream waits until a 32-bit word in device memory reaches a value / a
// stream writes such a word.  Used to let a copy-out stream start when a running kernel says its result is complete.
typedef CUresult (*StreamValueFn)(CUstream, CUdeviceptr, cuuint32_t, unsigned int);
StreamValueFn get_stream_value_fn(bool wait) {
  static StreamValueFn fns[2] = {nullptr, nullptr};
  static bool looked[2] = {false, false};
  if (!looked[wait]) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint(wait ? "cuStreamWaitValue32" : "cuStreamWriteValue32", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fns[wait] = reinterpret_cast<StreamValueFn>(p);
    looked[wait] = true;
  }
  return fns[wait];
}

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 tensor of `rank` dimensions (dims[0] innermost, strides in bytes for dims 1..), 128-byte
// swizzle, zero fill outside the tensor on loads, clipping on stores.
int encode_tiled(CUtensorMap* tm, const void* base, int rank, const uint64_t* dims, const uint64_t* strides,
                 const uint32_t* box, bool swizzle = true) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) {
    g_cuda_error = "cuTensorMapEncodeTiled entry point not available";
    return MOE_ERR_CUDA;
  }
  cuuint64_t gdim[5], gstr[4];
  cuuint32_t bx[5], estr[5] = {1, 1, 1, 1, 1};
  for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bx[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides[i];
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base), gdim, gstr, bx, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    char buf[200];
    snprintf(buf, sizeof buf, "cuTensorMapEncodeTiled failed (%d) rank=%d dims=%llu,%llu box=%u,%u", (int)r, rank,
             (unsigned long long)dims[0], (unsigned long long)dims[1], box[0], box[1]);
    g_cuda_error = buf;
    return MOE_ERR_CUDA;
  }
  return MOE_OK;
}

// Row-major [rows][cols] matrix, box [box_rows][box_cols].
int encode_2d(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
              uint32_t box_cols) {
  const uint64_t dims[2] = {cols, rows}, strides[1] = {cols * 2};
  const uint32_t box[2] = {box_cols, box_rows};
  return encode_tiled(tm, base, 2, dims, strides, box);
}

// Store map of a [rows][2][F] view of a [rows][2F] matrix (gate half, up half): box 32 rows x 64 columns
// of one half, so a column tile that ends past F is clipped instead of spilling into the other half.
int encode_halves(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t F) {
  const uint64_t dims[3] = {F, 2, rows}, strides[2] = {F * 2, 2 * F * 2};
  const uint32_t box[3] = {64, 1, 32};
  return encode_tiled(tm, base, 3, dims, strides, box);
}

// Store maps of the token-column tiles: un-swizzled boxes of 32 rows x `box_cols` columns.
int encode_2d_plain(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_cols) {
  const uint64_t dims[2] = {cols, rows}, strides[1] = {cols * 2};
  const uint32_t box[2] = {box_cols, 32};
  return encode_tiled(tm, base, 2, dims, strides, box, false);
}
int encode_halves_plain(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t F, uint32_t box_cols) {
  const uint64_t dims[3] = {F, 2, rows}, strides[2] = {F * 2, 2 * F * 2};
  const uint32_t box[3] = {box_cols, 1, 32};
  return encode_tiled(tm, base, 3, dims, strides, box, false);
}
// Load map of W_gate_up viewed as [Ep][F/16 groups][gate | up][16 rows][d]: one box brings, for four
// groups of 16 features, the 16 gate rows followed by the 16 up rows (needs F % 16 == 0).
int encode_gate_up_rows(CUtensorMap* tm, const void* base, uint64_t Ep, uint64_t F, uint64_t d) {
  const uint64_t dims[5] = {d, 16, 2, F / 16, Ep};
  const uint64_t strides[4] = {d * 2, F * d * 2, 16 * d * 2, 2 * F * d * 2};
  const uint32_t box[5] = {64, 16, 2, 4, 1};
  return encode_tiled(tm, base, 5, dims, strides, box);
}

// Store map of a weight-gradient tensor [Ep][M][N]: box 32 rows x 64 columns inside one expert slab.
int encode_slabs(CUtensorMap* tm, const void* base, uint64_t Ep, uint64_t M, uint64_t N) {
  const uint64_t dims[3] = {N, M, Ep}, strides[2] = {N * 2, M * N * 2};
  const uint32_t box[3] = {64, 32, 1};
  return encode_tiled(tm, base, 3, dims, strides, box);
}

bool shape_ok(const moe_shape* s) {
  return s && s->T_max >= 0 && s->d >= 8 && s->d % 8 == 0 && s->F >= 8 && s->F % 8 == 0 && s->E >= 1 &&
         s->E <= 1024 && s->k >= 1 && s->k <= s->E && s->k <= 32 && s->n_shared >= 0 && s->n_shared <= 64 &&
         (long)s->T_max * (s->k + s->n_shared) < (1l << 30);
}

constexpr int TRACE_RECORDS = 1 << 18;   // 32-byte records of the per-tile trace (MOE_FLAG_TRACE)

struct Carve {
  size_t off = 0;
  size_t take(size_t bytes) {
    size_t o = off;
    off += (bytes + 255) & ~size_t(255);
    return o;
  }
};

// Byte offsets of every workspace tensor.
struct WsPlan {
  size_t status, meta, counts, offsets, pad_off, mb_start, mblk_expert, pair_start, pblk_expert, work_start, wblk_expert, blk_hist, row_of, src_of, prow_of, combine_order, tok_last, prow_w,
      dw_partial, Xp, H, A, Y, dOutp, dH, st_x, st_dout, st_ids, st_w, st_out, st_dx, st_dw, st_logits, ctr, trace, total;
  int cap_rows, nblk_max, ntn_act, ctr_count, trace_cap;
};

WsPlan plan_workspace(const moe_shape& s) {
  WsPlan p;
  Carve c;
  const int Ep = s.E + s.n_shared, kp = s.k + s.n_shared;
  const size_t slots = (size_t)s.T_max * kp;
  p.cap_rows = padded_rows_max(s.T_max, kp, Ep);
  p.nblk_max = (int)((slots + LAYOUT_CHUNK - 1) / LAYOUT_CHUNK);
  if (p.nblk_max < 1) p.nblk_max = 1;
  p.ntn_act = (s.F + 255) / 256;
  const bool train = (s.flags & MOE_FLAG_SAVE_FOR_BWD) != 0;
  const size_t cap = (size_t)p.cap_rows;
  p.status = c.take(sizeof(DevStatus));
  p.meta = c.take(sizeof(int) * 8);
  p.counts = c.take(sizeof(int) * Ep);
  p.offsets = c.take(sizeof(int) * (Ep + 1));
  p.pad_off = c.take(sizeof(int) * (Ep + 1));
  p.mb_start = c.take(sizeof(int) * (Ep + 1));
  p.mblk_expert = c.take(sizeof(int) * (cap / BLOCK_M + 1));
  p.pair_start = c.take(sizeof(int) * (Ep + 1));
  p.pblk_expert = c.take(sizeof(int) * (cap / BLOCK_M + 1));
  p.work_start = c.take(sizeof(int) * (Ep + 1));
  p.wblk_expert = c.take(sizeof(int) * (cap / BLOCK_M + 1));
  p.blk_hist = c.take(sizeof(int) * (size_t)p.nblk_max * Ep);
  p.row_of = c.take(sizeof(int) * (slots + 1));
  p.src_of = c.take(sizeof(int) * (slots + 1));
  p.prow_of = c.take(sizeof(int) * (slots + 1));
  p.combine_order = c.take(sizeof(int) * ((size_t)s.T_max + 1));
  p.tok_last = c.take(sizeof(int) * ((size_t)s.T_max + 1));
  p.prow_w = c.take(sizeof(float) * cap);
  p.dw_partial = c.take(train ? sizeof(float) * cap * p.ntn_act * DW_PARTS_PER_TILE : 0);
  p.Xp = c.take(2 * cap * s.d);
  p.H = c.take(train ? 2 * cap * 2 * s.F : 0);
  p.A = c.take(2 * cap * s.F);
  p.Y = c.take(2 * cap * s.d);
  p.dOutp = c.take(train ? 2 * cap * s.d : 0);
  p.dH = c.take(train ? 2 * cap * 2 * s.F : 0);
  p.st_x = c.take(2 * (size_t)s.T_max * s.d);
  p.st_dout = c.take(train ? 2 * (size_t)s.T_max * s.d : 0);
  p.st_ids = c.take(sizeof(int) * (size_t)s.T_max * s.k);
  p.st_w = c.take(sizeof(float) * (size_t)s.T_max * s.k);
  p.st_out = c.take(2 * (size_t)s.T_max * s.d);
  p.st_dx = c.take(train ? 2 * (size_t)s.T_max * s.d : 0);   // its own buffer: a deferred copy of out may still read st_out
  p.st_dw = c.take(sizeof(float) * (size_t)s.T_max * s.k);
  p.st_logits = c.take(sizeof(float) * (size_t)s.T_max * s.E);
  p.ctr_count = ctr_ints((int)(cap / BLOCK_M) + 1);
  p.ctr = c.take(sizeof(int) * (size_t)p.ctr_count);
  p.trace_cap = (s.flags & MOE_FLAG_TRACE) ? TRACE_RECORDS : 0;
  p.trace = c.take((size_t)p.trace_cap * 32);
  p.total = c.off;
  return p;
}

}  // namespace

constexpr int HOST_CHUNKS = 4;   // token chunks of a host-buffer result (combine + copy-out pipelined)

struct moe_ctx {
  moe_shape shape;
  WsPlan plan;
  uint8_t* ws = nullptr;
  bool owns_ws = false;
  int device = 0;
  int num_sms = 0;
  int launches = 0;
  int saved_T = -1;  // T of the forward whose tensors are in the workspace (-1: none)
  const void *saved_x = nullptr, *saved_ids = nullptr, *saved_w = nullptr;  // that forward's inputs
  uint64_t budget_ns = 2000ull * 1000 * 1000;
  int dep_extra = 0;  // test hook: makes the activation dependencies of the persistent launch unreachable
  bool plain_launch = false;  // diagnostic: persistent launches without the cooperative attribute
  cudaStream_t last_stream = nullptr;
  // host-buffer entry points: a copy-in stream (the next call's large input arrives while the previous
  // call still computes) and a copy-out stream (the result leaves in token chunks behind the combine)
  bool copy_ready = false;
  cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
  cudaEvent_t ev_x_free = nullptr, ev_dout_free = nullptr, ev_h2d_done = nullptr, ev_d2h_done = nullptr, ev_out_done = nullptr;
  bool out_pending = false;   // MOE_FLAG_DEFER_OUT_COPY: the copy of the last forward's result may still be running
  cudaEvent_t ev_chunk[HOST_CHUNKS] = {};
  bool x_used = false, dout_used = false;
  // optional per-operator timing
  bool profiling = false;
  bool events_made = false;
  cudaEvent_t ev_start[MOE_NUM_PHASES], ev_stop[MOE_NUM_PHASES];
  bool phase_used[MOE_NUM_PHASES] = {};
  void begin_call(cudaStream_t st) {
    launches = 0;
    last_stream = st;
    for (bool& u : phase_used) u = false;
  }
  // tensor maps of workspace tensors (fixed for the context's lifetime)
  CUtensorMap tm_Xp_k, tm_A_k, tm_dOutp_k, tm_dH_k;      // K-major A operands, box 128 x 64
  CUtensorMap tm_dOutp_mn, tm_A_mn, tm_dH_mn, tm_Xp_mn;  // MN-major operands of the weight gradients, box 64 x 64
  // tensor maps of the caller's weights, re-encoded when the pointers change
  const void* w1_ptr = nullptr;
  const void* w2_ptr = nullptr;
  CUtensorMap tm_W1_k, tm_W2_k128, tm_W1_mn, tm_W2_mn;
  CUtensorMap tm_W1_gu;  // token-column tiles: 16 gate rows + 16 up rows per box
  // store maps: workspace tensors (fixed) and the caller's weight gradients (re-encoded on change)
  CUtensorMap ts_A, ts_H, ts_Y, ts_dH;
  // token-column tiles: token operands with 64-row and 16-row boxes, un-swizzled store maps
  CUtensorMap tk_Xp[8], tk_A[8], tk_dOutp[8], tk_dH[8];
  CUtensorMap tp_A, tp_H, tp_Y, tp_dH;
  const void* dw1_ptr = nullptr;
  const void* dw2_ptr = nullptr;
  CUtensorMap ts_dW1, ts_dW2;

  template <class T>
  T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
  DevStatus* status() const { return at<DevStatus>(plan.status); }
  LayoutView layout() const {
    LayoutView lv{};
    lv.counts = at<int>(plan.counts);
    lv.offsets = at<int>(plan.offsets);
    lv.row_of = at<int>(plan.row_of);
    lv.src_of = at<int>(plan.src_of);
    lv.prow_of = at<int>(plan.prow_of);
    lv.pad_off = at<int>(plan.pad_off);
    lv.mb_start = at<int>(plan.mb_start);
    lv.mblk_expert = at<int>(plan.mblk_expert);
    lv.pair_start = at<int>(plan.pair_start);
    lv.pblk_expert = at<int>(plan.pblk_expert);
    lv.work_start = at<int>(plan.work_start);
    lv.wblk_expert = at<int>(plan.wblk_expert);
    lv.meta = at<int>(plan.meta);
    lv.blk_hist = at<int>(plan.blk_hist);
    lv.combine_order = at<int>(plan.combine_order);
    lv.tok_last = (!(shape.flags & MOE_FLAG_SERIAL_LAUNCH) && shape.F % 16 == 0) ? at<int>(plan.tok_last) : nullptr;
    return lv;
  }
  Dims dims(int T) const { return Dims{T, shape.d, shape.E, shape.k, shape.n_shared, shape.F}; }
  bool train() const { return (shape.flags & MOE_FLAG_SAVE_FOR_BWD) != 0; }
};

namespace {

// Brackets one operator's launches with events when profiling is on.
struct Phase {
  moe_ctx* c;
  int id;
  cudaStream_t st;
  Phase(moe_ctx* c_, int id_, cudaStream_t st_) : c(c_), id(id_), st(st_) {
    if (c->profiling) cudaEventRecord(c->ev_start[id], st);
  }
  ~Phase() {
    if (c->profiling) {
      cudaEventRecord(c->ev_stop[id], st);
      c->phase_used[id] = true;
    }
  }
};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

int encode_weight_maps(moe_ctx* c, const uint16_t* W1, const uint16_t* W2) {
  const moe_shape& s = c->shape;
  const uint64_t Ep = s.E + s.n_shared;
  int rc;
  if (W1 != c->w1_ptr) {
    if ((rc = encode_2d(&c->tm_W1_k, W1, Ep * 2 * s.F, s.d, 128, 64))) return rc;
    if ((rc = encode_2d(&c->tm_W1_mn, W1, Ep * 2 * s.F, s.d, 64, 64))) return rc;
    if (s.F % 16 == 0 && (rc = encode_gate_up_rows(&c->tm_W1_gu, W1, Ep, s.F, s.d))) return rc;
    c->w1_ptr = W1;
  }
  if (W2 != c->w2_ptr) {
    if ((rc = encode_2d(&c->tm_W2_k128, W2, Ep * s.d, s.F, 128, 64))) return rc;
    if ((rc = encode_2d(&c->tm_W2_mn, W2, Ep * s.d, s.F, 64, 64))) return rc;
    c->w2_ptr = W2;
  }
  return MOE_OK;
}

GemmArgs base_args(const moe_ctx* c) {
  GemmArgs g;
  memset(&g, 0, sizeof g);
  LayoutView lv = c->layout();
  g.mblk_expert = lv.mblk_expert;
  g.mb_start = lv.mb_start;
  g.counts = lv.counts;
  g.meta = lv.meta;
  g.pair_start = lv.pair_start;
  g.pblk_expert = lv.pblk_expert;
  g.work_start = lv.work_start;
  g.wblk_expert = lv.wblk_expert;
  g.cap_rows = c->plan.cap_rows;
  g.Ep = c->shape.E + c->shape.n_shared;
  g.F = c->shape.F;
  g.status = c->status();
  g.budget_ns = c->budget_ns;
  return g;
}

// GMM1 + SwiGLU (+ routing weight): A = w * silu(Xp.Wg^T) * (Xp.Wu^T)
GemmArgs args_gate_up(const moe_ctx* c) {
  const moe_shape& s = c->shape;
  GemmArgs g = base_args(c);
  g.tmA = c->tm_Xp_k;
  g.tmB = c->tm_W1_k;
  g.n_tiles_n = (s.F + 127) / 128;
  g.K = s.d;
  g.N = s.F;
  g.b_rows_per_expert = 2 * s.F;
  g.tmOut0 = c->ts_A;
  g.tmOut1 = c->ts_H;
  g.save_h = c->train() ? 1 : 0;
  g.prow_w = c->at<float>(c->plan.prow_w);
  return g;
}
// GMM2: Y = A . W_down^T
GemmArgs args_down(const moe_ctx* c) {
  const moe_shape& s = c->shape;
  GemmArgs g = base_args(c);
  g.tmA = c->tm_A_k;
  g.tmB = c->tm_W2_k128;  // each CTA of a pair loads 128 of the tile's 256 rows
  g.n_tiles_n = (s.d + 255) / 256;
  g.K = s.F;
  g.N = s.d;
  g.b_rows_per_expert = s.d;
  g.tmOut0 = c->ts_Y;
  return g;
}
// act_grad + SwiGLU_grad (+ routing-weight gradient partials)
GemmArgs args_act_grad(const moe_ctx* c, bool want_dw) {
  const moe_shape& s = c->shape;
  const WsPlan& p = c->plan;
  GemmArgs g = base_args(c);
  g.tmA = c->tm_dOutp_k;
  g.tmB = c->tm_W2_mn;
  g.n_tiles_n = p.ntn_act;
  g.K = s.d;
  g.N = s.F;
  g.b_rows_per_expert = s.d;
  g.tmOut0 = c->ts_dH;
  g.in0 = c->at<uint16_t>(p.H);
  g.ld_in0 = 2 * s.F;
  g.prow_w = c->at<float>(p.prow_w);
  g.dw_partial = want_dw ? c->at<float>(p.dw_partial) : nullptr;
  return g;
}
// w2_grad: dW_down[e][c][f] = sum_rows dOutp[r][c] * A[r][f]   (shares dOutp with act_grad)
GemmArgs args_wgrad_down(const moe_ctx* c) {
  const moe_shape& s = c->shape;
  GemmArgs g = base_args(c);
  g.tmA = c->tm_dOutp_mn;
  g.tmB = c->tm_A_mn;
  g.M = s.d;
  g.N = s.F;
  g.n_tiles_m = (s.d + 127) / 128;
  g.n_tiles_n = (s.F + 255) / 256;
  g.tmOut0 = c->ts_dW2;
  return g;
}
// gate_grad: dXp = dH . W_gate_up[e]   (the forward's Y is dead by now: its buffer receives dXp)
GemmArgs args_gate_grad(const moe_ctx* c) {
  const moe_shape& s = c->shape;
  GemmArgs g = base_args(c);
  g.tmA = c->tm_dH_k;
  g.tmB = c->tm_W1_mn;
  g.n_tiles_n = (s.d + 255) / 256;
  g.K = 2 * s.F;
  g.N = s.d;
  g.b_rows_per_expert = 2 * s.F;
  g.tmOut0 = c->ts_Y;
  return g;
}
// w1_grad: dW_gate_up[e][n][c] = sum_rows dH[r][n] * Xp[r][c]   (shares dH with gate_grad)
GemmArgs args_wgrad_gate_up(const moe_ctx* c) {
  const moe_shape& s = c->shape;
  GemmArgs g = base_args(c);
  g.tmA = c->tm_dH_mn;
  g.tmB = c->tm_Xp_mn;
  g.M = 2 * s.F;
  g.N = s.d;
  g.n_tiles_m = (2 * s.F + 127) / 128;
  g.n_tiles_n = (s.d + 255) / 256;
  g.tmOut0 = c->ts_dW1;
  return g;
}

// Token-column tiles (gemm_tc3.cu, and the persistent launch) need the 16-feature gate/up groups of W_gate_up.
bool token_col_tiles(const moe_ctx* c) { return c->shape.F % 16 == 0; }
// Rewrites the arguments of a row-space operator for the token-column tiles: tmA/tmTok16 = tokens,
// tmB = weights, un-swizzled store maps.
GemmArgs to_token_cols(const moe_ctx* c, GemmMode mode, GemmArgs g) {
  switch (mode) {
    case GEMM_GATE_UP:
      g.tmA = c->tm_Xp_k; memcpy(g.tmTok, c->tk_Xp, sizeof g.tmTok); g.tmB = c->tm_W1_gu;
      g.tmOut0 = c->tp_A; g.tmOut1 = c->tp_H;
      break;
    case GEMM_DOWN:
      g.tmA = c->tm_A_k; memcpy(g.tmTok, c->tk_A, sizeof g.tmTok); g.tmB = c->tm_W2_k128;
      g.tmOut0 = c->tp_Y;
      break;
    case GEMM_ACT_GRAD:
      g.tmA = c->tm_dOutp_k; memcpy(g.tmTok, c->tk_dOutp, sizeof g.tmTok);
      g.tmOut0 = c->tp_dH;
      break;
    case GEMM_GATE_GRAD:
      g.tmA = c->tm_dH_k; memcpy(g.tmTok, c->tk_dH, sizeof g.tmTok);
      g.tmOut0 = c->tp_Y;
      break;
    default: break;
  }
  return g;
}
cudaError_t launch_gemm_serial(const moe_ctx* c, GemmMode mode, const GemmArgs& args, cudaStream_t st, int* launches) {
  if (mode == GEMM_WGRAD) return launch_wgrad_strips(args, c->num_sms, st, launches);
  if (token_col_tiles(c)) return launch_gemm3(mode, to_token_cols(c, mode, args), c->num_sms, st, launches);
  return launch_gemm2(mode, args, c->num_sms, st, launches);
}
#define LAUNCH_GEMM_SERIAL(mode, args, sms, st, launches) launch_gemm_serial(c, mode, args, st, launches)

// One launch per operator: on request, and for shapes the persistent launch does not cover (it runs the
// token-column tiles only).
int gate_mode(const moe_ctx* c) {
  return ((c->shape.flags & MOE_FLAG_RENORM_TOPK) ? GATE_RENORM : 0) | ((c->shape.flags & MOE_FLAG_SIGMOID_GATE) ? GATE_SIGMOID : 0);
}
bool serial_mode(const moe_ctx* c) { return (c->shape.flags & MOE_FLAG_SERIAL_LAUNCH) != 0 || !token_col_tiles(c); }

ChainParams chain_params(const moe_ctx* c, bool bwd, int T, bool want_dw) {
  const moe_shape& s = c->shape;
  ChainParams cp;
  memset(&cp, 0, sizeof cp);
  cp.is_bwd = bwd ? 1 : 0;
  cp.Ep = s.E + s.n_shared;
  cp.T = T;
  cp.k = s.k;
  cp.kp = s.k + s.n_shared;
  cp.dep_extra = c->dep_extra;
  cp.want_dw = want_dw ? 1 : 0;
  if (!bwd) {
    cp.n_phases = 2;
    cp.ntn[0] = (s.F + 127) / 128;                 // gate+up: 128 features (gate and up) per pair tile
    cp.ntn[1] = (s.d + 255) / 256;                 // down
    cp.merges[1] = 1;
  } else {
    cp.n_phases = 4;
    cp.ntn[0] = c->plan.ntn_act;                   // act_grad
    cp.ntn[1] = (s.F + 255) / 256;                 // w2_grad: column tiles per strip
    cp.strips[1] = (s.d + 255) / 256;
    cp.ntn[2] = (s.d + 255) / 256;                 // gate_grad
    cp.merges[2] = 1;
    cp.ntn[3] = (s.d + 255) / 256;                 // w1_grad
    cp.strips[3] = (2 * s.F + 255) / 256;
  }
  return cp;
}

FusedArgs fused_base(moe_ctx* c, bool bwd, int T) {
  const moe_shape& s = c->shape;
  const WsPlan& p = c->plan;
  FusedArgs fa;
  memset(&fa, 0, sizeof fa);
  fa.lv = c->layout();
  fa.ctr = c->at<int>(p.ctr);
  fa.d = s.d;
  fa.kp = s.k + s.n_shared;
  fa.trace = p.trace_cap ? c->at<uint4>(p.trace) : nullptr;
  fa.trace_cap = p.trace_cap;
  fa.status = c->status();
  fa.budget_ns = c->budget_ns;
  return fa;
}

int ensure_copy_streams(moe_ctx* c) {
  if (c->copy_ready) return MOE_OK;
  MOE_CUDA(cudaStreamCreateWithFlags(&c->h2d_stream, cudaStreamNonBlocking));
  MOE_CUDA(cudaStreamCreateWithFlags(&c->d2h_stream, cudaStreamNonBlocking));
  cudaEvent_t* evs[] = {&c->ev_x_free, &c->ev_dout_free, &c->ev_h2d_done, &c->ev_d2h_done, &c->ev_out_done};
  for (cudaEvent_t* e : evs) MOE_CUDA(cudaEventCreateWithFlags(e, cudaEventDisableTiming));
  for (int i = 0; i < HOST_CHUNKS; ++i) MOE_CUDA(cudaEventCreateWithFlags(&c->ev_chunk[i], cudaEventDisableTiming));
  c->copy_ready = true;
  return MOE_OK;
}

// The forward result leaves for the host: on `st`, or -- MOE_FLAG_DEFER_OUT_COPY -- on the copy-out stream behind an
// event, so that it overlaps whatever the caller enqueues on `st` next; join_out_copy() makes `st` cover it later.
int copy_out_to_host(moe_ctx* c, const uint16_t* out, uint16_t* out_host, size_t bytes, cudaStream_t st) {
  if (!(c->shape.flags & MOE_FLAG_DEFER_OUT_COPY)) {
    MOE_CUDA(cudaMemcpyAsync(out_host, out, bytes, cudaMemcpyDeviceToHost, st));
    return MOE_OK;
  }
  MOE_CUDA(cudaEventRecord(c->ev_chunk[1], st));
  MOE_CUDA(cudaStreamWaitEvent(c->d2h_stream, c->ev_chunk[1], 0));
  MOE_CUDA(cudaMemcpyAsync(out_host, out, bytes, cudaMemcpyDeviceToHost, c->d2h_stream));
  MOE_CUDA(cudaEventRecord(c->ev_out_done, c->d2h_stream));
  c->out_pending = true;
  return MOE_OK;
}
int join_out_copy(moe_ctx* c, cudaStream_t st) {
  if (!c->out_pending) return MOE_OK;
  MOE_CUDA(cudaStreamWaitEvent(st, c->ev_out_done, 0));
  c->out_pending = false;
  return MOE_OK;
}

// Combine into `out` (device).  With `out_host` the tokens are combined in HOST_CHUNKS launches and
// each chunk is copied out on the copy-out stream while the next one is being combined; the
// launching stream then waits for the last copy, so the host buffer is complete once `st` is.
int combine_and_maybe_copy_out(moe_ctx* c, const Dims& dm, const LayoutView& lv, uint16_t* out, uint16_t* out_host,
                               cudaStream_t st) {
  const WsPlan& p = c->plan;
  if (!out_host || dm.T < HOST_CHUNKS * 64) {
    MOE_CUDA(launch_combine(c->at<uint16_t>(p.Y), dm, lv, out, st, &c->launches));
    if (out_host) return copy_out_to_host(c, out, out_host, 2 * (size_t)dm.T * dm.d, st);
    return MOE_OK;
  }
  for (int i = 0; i < HOST_CHUNKS; ++i) {
    const int t0 = (int)((long)dm.T * i / HOST_CHUNKS), t1 = (int)((long)dm.T * (i + 1) / HOST_CHUNKS);
    MOE_CUDA(launch_combine(c->at<uint16_t>(p.Y), dm, lv, out, st, &c->launches, t0, t1));
    MOE_CUDA(cudaEventRecord(c->ev_chunk[i], st));
    MOE_CUDA(cudaStreamWaitEvent(c->d2h_stream, c->ev_chunk[i], 0));
    MOE_CUDA(cudaMemcpyAsync(out_host + (size_t)t0 * dm.d, out + (size_t)t0 * dm.d, 2 * (size_t)(t1 - t0) * dm.d,
                             cudaMemcpyDeviceToHost, c->d2h_stream));
  }
  if (c->shape.flags & MOE_FLAG_DEFER_OUT_COPY) {   // the caller lets the copy run behind what it enqueues next
    MOE_CUDA(cudaEventRecord(c->ev_out_done, c->d2h_stream));
    c->out_pending = true;
    return MOE_OK;
  }
  MOE_CUDA(cudaEventRecord(c->ev_d2h_done, c->d2h_stream));
  MOE_CUDA(cudaStreamWaitEvent(st, c->ev_d2h_done, 0));
  return MOE_OK;
}

int run_fwd(moe_ctx* c, const uint16_t* x, const int32_t* ids, const float* w, const uint16_t* W1,
            const uint16_t* W2, uint16_t* out, int T, cudaStream_t st, uint16_t* out_host = nullptr) {
  const WsPlan& p = c->plan;
  const Dims dm = c->dims(T);
  const LayoutView lv = c->layout();
  int rc = encode_weight_maps(c, W1, W2);
  if (rc) return rc;
  c->saved_T = -1;
  {
    Phase ph(c, MOE_PHASE_LAYOUT, st);
    MOE_CUDA(launch_layout(ids, dm, lv, c->status(), st, &c->launches));
    // with shared experts every token's last row belongs to the last expert: token order is as good as any
    if (!serial_mode(c)) MOE_CUDA(launch_layout_order(dm, lv, p.cap_rows / BLOCK_M, st, &c->launches));
  }
  if (serial_mode(c)) {
    {
      Phase ph(c, MOE_PHASE_GATHER, st);
      MOE_CUDA(launch_gather(x, w, dm, lv, c->at<uint16_t>(p.Xp), c->at<float>(p.prow_w), p.cap_rows, st,
                             &c->launches, c->status(), c->budget_ns));
    }
    {
      Phase ph(c, MOE_PHASE_GEMM_GATE_UP, st);
      MOE_CUDA(LAUNCH_GEMM_SERIAL(GEMM_GATE_UP, args_gate_up(c), c->num_sms, st, &c->launches));
    }
    {
      Phase ph(c, MOE_PHASE_GEMM_DOWN, st);
      MOE_CUDA(LAUNCH_GEMM_SERIAL(GEMM_DOWN, args_down(c), c->num_sms, st, &c->launches));
    }
    {
      Phase ph(c, MOE_PHASE_COMBINE, st);
      if ((rc = combine_and_maybe_copy_out(c, dm, lv, out, out_host, st))) return rc;
    }
  } else {
    // one persistent launch: gather, GMM1+SwiGLU, GMM2 and combine tiles ordered by event counters
    FusedArgs fa = fused_base(c, false, T);
    fa.cp = chain_params(c, false, T, false);
    fa.op[0] = to_token_cols(c, GEMM_GATE_UP, args_gate_up(c));
    fa.op[1] = to_token_cols(c, GEMM_DOWN, args_down(c));
    fa.gather_src = x;
    fa.gather_dst = c->at<uint16_t>(p.Xp);
    fa.topk_w = w;
    fa.prow_w = c->at<float>(p.prow_w);
    fa.combine_rows = c->at<uint16_t>(p.Y);
    fa.combine_out = out;
    Phase ph(c, MOE_PHASE_FUSED_FWD, st);
    MOE_CUDA(cudaMemsetAsync(fa.ctr, 0, sizeof(int) * (size_t)p.ctr_count, st));
    MOE_CUDA(launch_fused(false, fa, c->num_sms, !c->plain_launch, st, &c->launches));
    if (out_host && (rc = copy_out_to_host(c, out, out_host, 2 * (size_t)T * c->shape.d, st))) return rc;
  }
  if (c->train()) {
    c->saved_T = T;
    c->saved_x = x; c->saved_ids = ids; c->saved_w = w;
  }
  return MOE_OK;
}

int run_bwd(moe_ctx* c, const uint16_t* dout, const uint16_t* W1, const uint16_t* W2, uint16_t* dx, uint16_t* dW1,
            uint16_t* dW2, float* d_w, int T, cudaStream_t st, uint16_t* dx_host = nullptr) {
  const moe_shape& s = c->shape;
  const WsPlan& p = c->plan;
  const Dims dm = c->dims(T);
  const LayoutView lv = c->layout();
  int rc = encode_weight_maps(c, W1, W2);
  if (rc) return rc;
  const uint64_t Ep = s.E + s.n_shared;
  if (dW1 != c->dw1_ptr) {
    if ((rc = encode_slabs(&c->ts_dW1, dW1, Ep, 2 * s.F, s.d))) return rc;
    c->dw1_ptr = dW1;
  }
  if (dW2 != c->dw2_ptr) {
    if ((rc = encode_slabs(&c->ts_dW2, dW2, Ep, s.d, s.F))) return rc;
    c->dw2_ptr = dW2;
  }
  if (serial_mode(c)) {
    {  // backward Dispatch: expert-ordered gather of the upstream gradient
      Phase ph(c, MOE_PHASE_BWD_GATHER, st);
      MOE_CUDA(launch_gather(dout, nullptr, dm, lv, c->at<uint16_t>(p.dOutp), nullptr, p.cap_rows, st,
                             &c->launches, c->status(), c->budget_ns));
    }
    {
      Phase ph(c, MOE_PHASE_ACT_GRAD, st);
      MOE_CUDA(LAUNCH_GEMM_SERIAL(GEMM_ACT_GRAD, args_act_grad(c, d_w != nullptr), c->num_sms, st, &c->launches));
    }
    if (d_w) {
      Phase ph(c, MOE_PHASE_DW_REDUCE, st);
      MOE_CUDA(launch_dw_reduce(c->at<float>(p.dw_partial), token_col_tiles(c) ? p.ntn_act * DW_PARTS_PER_TILE : p.ntn_act,
                                dm, lv, d_w, st, &c->launches));
    }
    {
      Phase ph(c, MOE_PHASE_WGRAD_DOWN, st);
      MOE_CUDA(LAUNCH_GEMM_SERIAL(GEMM_WGRAD, args_wgrad_down(c), c->num_sms, st, &c->launches));
    }
    {
      Phase ph(c, MOE_PHASE_GATE_GRAD, st);
      MOE_CUDA(LAUNCH_GEMM_SERIAL(GEMM_GATE_GRAD, args_gate_grad(c), c->num_sms, st, &c->launches));
    }
    {  // backward Combine: before the last weight gradient, which does not need dXp, so that with
       // host buffers the copy of dx leaves on the copy-out stream while that GEMM runs
      Phase ph(c, MOE_PHASE_BWD_COMBINE, st);
      MOE_CUDA(launch_combine(c->at<uint16_t>(p.Y), dm, lv, dx, st, &c->launches));
      if (dx_host) {
        MOE_CUDA(cudaEventRecord(c->ev_chunk[0], st));
        MOE_CUDA(cudaStreamWaitEvent(c->d2h_stream, c->ev_chunk[0], 0));
        MOE_CUDA(cudaMemcpyAsync(dx_host, dx, 2 * (size_t)T * s.d, cudaMemcpyDeviceToHost, c->d2h_stream));
        MOE_CUDA(cudaEventRecord(c->ev_d2h_done, c->d2h_stream));
      }
    }
    {
      Phase ph(c, MOE_PHASE_WGRAD_GATE_UP, st);
      MOE_CUDA(LAUNCH_GEMM_SERIAL(GEMM_WGRAD, args_wgrad_gate_up(c), c->num_sms, st, &c->launches));
    }
    if (dx_host) MOE_CUDA(cudaStreamWaitEvent(st, c->ev_d2h_done, 0));  // dx_host is complete once `st` is
  } else {
    FusedArgs fa = fused_base(c, true, T);
    fa.cp = chain_params(c, true, T, d_w != nullptr);
    fa.op[0] = to_token_cols(c, GEMM_ACT_GRAD, args_act_grad(c, d_w != nullptr));
    fa.op[1] = args_wgrad_down(c);
    fa.op[2] = to_token_cols(c, GEMM_GATE_GRAD, args_gate_grad(c));
    fa.op[3] = args_wgrad_gate_up(c);
    fa.gather_src = dout;
    fa.gather_dst = c->at<uint16_t>(p.dOutp);
    fa.combine_rows = c->at<uint16_t>(p.Y);
    fa.combine_out = dx;
    fa.dw_partial = c->at<float>(p.dw_partial);
    fa.dw_nparts = p.ntn_act * DW_PARTS_PER_TILE;
    fa.d_topk_w = d_w;
    Phase ph(c, MOE_PHASE_FUSED_BWD, st);
    MOE_CUDA(cudaMemsetAsync(fa.ctr, 0, sizeof(int) * (size_t)p.ctr_count, st));
    // slots dropped for an invalid expert id have no row: their gradient is zero
    if (d_w) MOE_CUDA(cudaMemsetAsync(d_w, 0, sizeof(float) * (size_t)T * s.k, st));
    // Host buffers: dx is complete when the last backward-combine task is, well before the last weight-gradient
    // strips; the kernel then sets a word the copy-out stream waits for, so the copy overlaps the rest of the launch.
    StreamValueFn wait_value = dx_host ? get_stream_value_fn(true) : nullptr;
    StreamValueFn write_value = dx_host ? get_stream_value_fn(false) : nullptr;
    const bool early_out = wait_value && write_value;
    const CUdeviceptr ready_word = reinterpret_cast<CUdeviceptr>(fa.ctr + CTR_OUT_READY);
    fa.announce_out = early_out ? 1 : 0;
    if (early_out) {
      MOE_CUDA(cudaEventRecord(c->ev_chunk[0], st));   // the word is cleared (the memset above) before anyone waits on it
      MOE_CUDA(cudaStreamWaitEvent(c->d2h_stream, c->ev_chunk[0], 0));
      if (wait_value(c->d2h_stream, ready_word, 1, CU_STREAM_WAIT_VALUE_GEQ) != CUDA_SUCCESS) return cuda_fail(cudaErrorUnknown, "cuStreamWaitValue32");
      MOE_CUDA(cudaMemcpyAsync(dx_host, dx, 2 * (size_t)T * s.d, cudaMemcpyDeviceToHost, c->d2h_stream));
      MOE_CUDA(cudaEventRecord(c->ev_d2h_done, c->d2h_stream));
    }
    const cudaError_t launched = launch_fused(true, fa, c->num_sms, !c->plain_launch, st, &c->launches);
    if (early_out) {
      // a launch that failed, or gave up on an expired wait, never sets the word: set it behind the launch so that
      // the copy-out stream is released in every case, then make `st` cover the copy
      if (write_value(st, ready_word, 1, CU_STREAM_WRITE_VALUE_DEFAULT) != CUDA_SUCCESS) return cuda_fail(cudaErrorUnknown, "cuStreamWriteValue32");
      MOE_CUDA(cudaStreamWaitEvent(st, c->ev_d2h_done, 0));
    }
    MOE_CUDA(launched);
    if (!early_out && dx_host) {
      MOE_CUDA(cudaMemcpyAsync(dx_host, dx, 2 * (size_t)T * s.d, cudaMemcpyDeviceToHost, st));
    }
  }
  return MOE_OK;
}

}  // namespace

extern "C" {

size_t moe_workspace_bytes(const moe_shape* shape) {
  if (!shape_ok(shape)) return 0;
  return plan_workspace(*shape).total;
}

int moe_create(moe_ctx** out, const moe_shape* shape, void* workspace, size_t workspace_bytes) {
  if (!out || !shape_ok(shape)) return MOE_ERR_INVALID_ARG;
  *out = nullptr;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return MOE_ERR_NO_DEVICE;
  }
  int major = 0, sms = 0;
  MOE_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  MOE_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  if (major != 10) return MOE_ERR_NO_DEVICE;
  moe_ctx* c = new moe_ctx();
  c->shape = *shape;
  c->plan = plan_workspace(*shape);
  c->device = dev;
  c->num_sms = sms;
  if (workspace) {
    if (workspace_bytes < c->plan.total || (reinterpret_cast<uintptr_t>(workspace) & 255)) {
      delete c;
      return MOE_ERR_WORKSPACE;
    }
    c->ws = static_cast<uint8_t*>(workspace);
  } else {
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&c->ws), c->plan.total);
    if (e != cudaSuccess) {
      delete c;
      return cuda_fail(e, "cudaMalloc(workspace)");
    }
    c->owns_ws = true;
  }
  const moe_shape& s = c->shape;
  const WsPlan& p = c->plan;
  const uint64_t cap = p.cap_rows;
  const bool train = c->train();
  int rc = MOE_OK;
  cudaError_t e = cudaMemset(c->ws, 0, p.Xp);  // status, tables and small arrays start at zero
  if (e != cudaSuccess) rc = cuda_fail(e, "cudaMemset(workspace)");
  if (!rc) rc = encode_2d(&c->tm_Xp_k, c->ws + p.Xp, cap, s.d, 128, 64);
  if (!rc) rc = encode_2d(&c->tm_A_k, c->ws + p.A, cap, s.F, 128, 64);
  if (!rc) rc = encode_2d(&c->ts_A, c->ws + p.A, cap, s.F, 32, 64);
  if (!rc) rc = encode_2d(&c->ts_Y, c->ws + p.Y, cap, s.d, 32, 64);
  if (!rc && train) rc = encode_halves(&c->ts_H, c->ws + p.H, cap, s.F);
  if (!rc && train) rc = encode_halves(&c->ts_dH, c->ws + p.dH, cap, s.F);
  if (!rc && train) rc = encode_2d(&c->tm_dOutp_k, c->ws + p.dOutp, cap, s.d, 128, 64);
  if (!rc && train) rc = encode_2d(&c->tm_dH_k, c->ws + p.dH, cap, 2 * s.F, 128, 64);
  if (!rc && train) rc = encode_2d(&c->tm_dOutp_mn, c->ws + p.dOutp, cap, s.d, 64, 64);
  if (!rc && train) rc = encode_2d(&c->tm_A_mn, c->ws + p.A, cap, s.F, 64, 64);
  if (!rc && train) rc = encode_2d(&c->tm_dH_mn, c->ws + p.dH, cap, 2 * s.F, 64, 64);
  if (!rc && train) rc = encode_2d(&c->tm_Xp_mn, c->ws + p.Xp, cap, s.d, 64, 64);
  for (int i = 0; i < 8 && !rc; ++i) {
    const uint32_t br = 16u * (i + 1);
    rc = encode_2d(&c->tk_Xp[i], c->ws + p.Xp, cap, s.d, br, 64);
    if (!rc) rc = encode_2d(&c->tk_A[i], c->ws + p.A, cap, s.F, br, 64);
    if (!rc && train) rc = encode_2d(&c->tk_dOutp[i], c->ws + p.dOutp, cap, s.d, br, 64);
    if (!rc && train) rc = encode_2d(&c->tk_dH[i], c->ws + p.dH, cap, 2 * s.F, br, 64);
  }
  if (!rc) rc = encode_2d_plain(&c->tp_A, c->ws + p.A, cap, s.F, 16);
  if (!rc) rc = encode_2d_plain(&c->tp_Y, c->ws + p.Y, cap, s.d, 32);
  if (!rc && train) rc = encode_halves_plain(&c->tp_H, c->ws + p.H, cap, s.F, 16);
  if (!rc && train) rc = encode_halves_plain(&c->tp_dH, c->ws + p.dH, cap, s.F, 32);
  if (rc) {
    if (c->owns_ws) cudaFree(c->ws);
    delete c;
    return rc;
  }
  *out = c;
  return MOE_OK;
}

int moe_destroy(moe_ctx* c) {
  if (!c) return MOE_OK;
  if (c->events_made)
    for (int i = 0; i < MOE_NUM_PHASES; ++i) {
      cudaEventDestroy(c->ev_start[i]);
      cudaEventDestroy(c->ev_stop[i]);
    }
  if (c->copy_ready) {
    cudaStreamSynchronize(c->h2d_stream);
    cudaStreamSynchronize(c->d2h_stream);
    cudaStreamDestroy(c->h2d_stream);
    cudaStreamDestroy(c->d2h_stream);
    cudaEventDestroy(c->ev_x_free);
    cudaEventDestroy(c->ev_dout_free);
    cudaEventDestroy(c->ev_h2d_done);
    cudaEventDestroy(c->ev_d2h_done);
    for (int i = 0; i < HOST_CHUNKS; ++i) cudaEventDestroy(c->ev_chunk[i]);
  }
  if (c->owns_ws) cudaFree(c->ws);
  delete c;
  return MOE_OK;
}

int moe_route(moe_ctx* c, const float* logits, int32_t T, int32_t* topk_ids, float* topk_w, int32_t* counts,
              void* stream) {
  if (!c || !logits || !topk_ids || !topk_w || T < 0 || T > c->shape.T_max) return MOE_ERR_INVALID_ARG;
  c->begin_call(static_cast<cudaStream_t>(stream));
  Phase ph(c, MOE_PHASE_ROUTE, c->last_stream);
  MOE_CUDA(launch_route(logits, T, c->shape.E, c->shape.k, gate_mode(c), topk_ids,
                        topk_w, counts, c->last_stream, &c->launches));
  return MOE_OK;
}

int moe_router_fwd(moe_ctx* c, const uint16_t* x, const uint16_t* W_r, int32_t T, int32_t* topk_ids, float* topk_w,
                   float* logits, int32_t* counts, void* stream) {
  if (!c || !x || !W_r || !topk_ids || !topk_w || T < 0 || T > c->shape.T_max) return MOE_ERR_INVALID_ARG;
  const moe_shape& s = c->shape;
  if (s.E > 256 || s.k > 8) return MOE_ERR_TOO_LARGE;
  if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(W_r)) & 15) return MOE_ERR_INVALID_ARG;
  if (logits && (reinterpret_cast<uintptr_t>(logits) & 15)) return MOE_ERR_INVALID_ARG;
  c->begin_call(static_cast<cudaStream_t>(stream));
  if (T == 0) return MOE_OK;
  RouterArgs a;
  memset(&a, 0, sizeof a);
  a.T = T; a.E = s.E; a.k = s.k; a.d = s.d;
  a.N = ((s.E + 15) / 16) * 16;
  if (a.N < 32) a.N = 32;
  a.renorm = gate_mode(c);
  a.topk_ids = topk_ids; a.topk_w = topk_w; a.logits = logits; a.counts = counts;
  a.status = c->status();
  a.budget_ns = c->budget_ns;
  int rc = encode_2d(&a.tmX, x, (uint64_t)T, (uint64_t)s.d, 128, 64);   // 128 token rows x one 64-wide k-block
  if (rc) return rc;
  if ((rc = encode_2d(&a.tmW, W_r, (uint64_t)s.E, (uint64_t)s.d, (uint32_t)(a.N / 2), 64))) return rc;
  Phase ph(c, MOE_PHASE_ROUTE, c->last_stream);
  MOE_CUDA(launch_router_fwd(a, c->num_sms, c->last_stream, &c->launches));
  return MOE_OK;
}

int moe_router_bwd(moe_ctx* c, const float* logits, const int32_t* topk_ids, const float* d_topk_w, int32_t T,
                   float* d_logits, void* stream) {
  if (!c || !logits || !topk_ids || !d_topk_w || !d_logits || T < 0 || T > c->shape.T_max) return MOE_ERR_INVALID_ARG;
  const moe_shape& s = c->shape;
  if (s.k > 32) return MOE_ERR_TOO_LARGE;
  c->begin_call(static_cast<cudaStream_t>(stream));
  MOE_CUDA(launch_router_bwd(logits, topk_ids, d_topk_w, T, s.E, s.k, gate_mode(c), d_logits,
                             c->last_stream, &c->launches));
  return MOE_OK;
}

int moe_route_host(moe_ctx* c, const float* logits_host, int32_t T, int32_t* topk_ids_host, float* topk_w_host,
                   void* stream) {
  if (!c || !logits_host || !topk_ids_host || !topk_w_host || T < 0 || T > c->shape.T_max)
    return MOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  c->begin_call(st);
  if (T == 0) return MOE_OK;
  const moe_shape& s = c->shape;
  const WsPlan& p = c->plan;
  MOE_CUDA(cudaMemcpyAsync(c->ws + p.st_logits, logits_host, sizeof(float) * (size_t)T * s.E,
                           cudaMemcpyHostToDevice, st));
  {
    Phase ph(c, MOE_PHASE_ROUTE, st);
    MOE_CUDA(launch_route(c->at<float>(p.st_logits), T, s.E, s.k, gate_mode(c),
                          c->at<int32_t>(p.st_ids), c->at<float>(p.st_w), nullptr, st, &c->launches));
  }
  MOE_CUDA(cudaMemcpyAsync(topk_ids_host, c->ws + p.st_ids, sizeof(int) * (size_t)T * s.k, cudaMemcpyDeviceToHost,
                           st));
  MOE_CUDA(cudaMemcpyAsync(topk_w_host, c->ws + p.st_w, sizeof(float) * (size_t)T * s.k, cudaMemcpyDeviceToHost,
                           st));
  return MOE_OK;
}

int moe_layout(moe_ctx* c, const int32_t* topk_ids, int32_t T, int32_t* counts, int32_t* offsets, int32_t* row_of,
               int32_t* src_of, void* stream) {
  if (!c || !topk_ids || T < 0 || T > c->shape.T_max) return MOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  c->begin_call(st);
  c->saved_T = -1;
  const Dims dm = c->dims(T);
  const LayoutView lv = c->layout();
  MOE_CUDA(launch_layout(topk_ids, dm, lv, c->status(), st, &c->launches));
  const size_t n = (size_t)dm.slots(), Ep = dm.Ep();
  if (counts) MOE_CUDA(cudaMemcpyAsync(counts, lv.counts, sizeof(int) * Ep, cudaMemcpyDeviceToDevice, st));
  if (offsets) MOE_CUDA(cudaMemcpyAsync(offsets, lv.offsets, sizeof(int) * (Ep + 1), cudaMemcpyDeviceToDevice, st));
  if (row_of && n) MOE_CUDA(cudaMemcpyAsync(row_of, lv.row_of, sizeof(int) * n, cudaMemcpyDeviceToDevice, st));
  if (src_of && n) MOE_CUDA(cudaMemcpyAsync(src_of, lv.src_of, sizeof(int) * n, cudaMemcpyDeviceToDevice, st));
  return MOE_OK;
}

int moe_ffn_fwd(moe_ctx* c, const uint16_t* x, const int32_t* topk_ids, const float* topk_w,
                const uint16_t* W_gate_up, const uint16_t* W_down, uint16_t* out, int32_t T, void* stream) {
  if (!c || T < 0 || T > c->shape.T_max) return MOE_ERR_INVALID_ARG;
  c->begin_call(static_cast<cudaStream_t>(stream));
  if (T == 0) return MOE_OK;  // nothing to compute; tensor pointers of an empty batch may be NULL
  if (!x || !topk_ids || !topk_w || !W_gate_up || !W_down || !out) return MOE_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(W_gate_up) || !aligned16(W_down) || !aligned16(out)) return MOE_ERR_INVALID_ARG;
  return run_fwd(c, x, topk_ids, topk_w, W_gate_up, W_down, out, T, c->last_stream);
}

int moe_ffn_bwd(moe_ctx* c, const uint16_t* dout, const uint16_t* x, const int32_t* topk_ids, const float* topk_w,
                const uint16_t* W_gate_up, const uint16_t* W_down, uint16_t* dx, uint16_t* dW_gate_up,
                uint16_t* dW_down, float* d_topk_w, int32_t T, void* stream) {
  if (!c || !dout || !x || !topk_ids || !topk_w || !W_gate_up || !W_down || !dx || !dW_gate_up || !dW_down ||
      T < 0 || T > c->shape.T_max)
    return MOE_ERR_INVALID_ARG;
  if (!aligned16(dout) || !aligned16(W_gate_up) || !aligned16(W_down) || !aligned16(dx) ||
      !aligned16(dW_gate_up) || !aligned16(dW_down))
    return MOE_ERR_INVALID_ARG;
  if (!c->train()) return MOE_ERR_STATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  c->begin_call(st);
  if (T == 0) {
    const moe_shape& s = c->shape;
    const size_t Ep = s.E + s.n_shared;
    MOE_CUDA(cudaMemsetAsync(dW_gate_up, 0, 2 * Ep * 2 * s.F * s.d, st));
    MOE_CUDA(cudaMemsetAsync(dW_down, 0, 2 * Ep * s.d * s.F, st));
    return MOE_OK;
  }
  // the backward works from what the forward saved: it must be the forward of these very tensors
  if (c->saved_T != T || c->saved_x != x || c->saved_ids != topk_ids || c->saved_w != topk_w) return MOE_ERR_STATE;
  return run_bwd(c, dout, W_gate_up, W_down, dx, dW_gate_up, dW_down, d_topk_w, T, st);
}

int moe_ffn_fwd_host(moe_ctx* c, const uint16_t* x_host, const int32_t* topk_ids_host, const float* topk_w_host,
                     const uint16_t* W_gate_up, const uint16_t* W_down, uint16_t* out_host, int32_t T,
                     void* stream) {
  if (!c || !x_host || !topk_ids_host || !topk_w_host || !W_gate_up || !W_down || !out_host || T < 0 ||
      T > c->shape.T_max)
    return MOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  c->begin_call(st);
  if (T == 0) return MOE_OK;
  const moe_shape& s = c->shape;
  const WsPlan& p = c->plan;
  int rc = ensure_copy_streams(c);
  if (rc) return rc;
  if ((rc = join_out_copy(c, st))) return rc;   // a deferred copy of the previous result still reads the staging buffer
  // x goes in on the copy-in stream as soon as the previous forward has read its staging buffer:
  // it overlaps whatever this context's earlier calls still have running on `st`
  if (c->x_used) MOE_CUDA(cudaStreamWaitEvent(c->h2d_stream, c->ev_x_free, 0));
  MOE_CUDA(cudaMemcpyAsync(c->ws + p.st_x, x_host, 2 * (size_t)T * s.d, cudaMemcpyHostToDevice, c->h2d_stream));
  MOE_CUDA(cudaEventRecord(c->ev_h2d_done, c->h2d_stream));
  MOE_CUDA(cudaMemcpyAsync(c->ws + p.st_ids, topk_ids_host, sizeof(int) * (size_t)T * s.k, cudaMemcpyHostToDevice,
                           st));
  MOE_CUDA(cudaMemcpyAsync(c->ws + p.st_w, topk_w_host, sizeof(float) * (size_t)T * s.k, cudaMemcpyHostToDevice,
                           st));
  MOE_CUDA(cudaStreamWaitEvent(st, c->ev_h2d_done, 0));
  rc = run_fwd(c, c->at<uint16_t>(p.st_x), c->at<int32_t>(p.st_ids), c->at<float>(p.st_w), W_gate_up, W_down,
               c->at<uint16_t>(p.st_out), T, st, out_host);
  if (rc) return rc;
  MOE_CUDA(cudaEventRecord(c->ev_x_free, st));
  c->x_used = true;
  return MOE_OK;
}

int moe_ffn_bwd_host(moe_ctx* c, const uint16_t* dout_host, const uint16_t* W_gate_up, const uint16_t* W_down,
                     uint16_t* dx_host, uint16_t* dW_gate_up, uint16_t* dW_down, float* d_topk_w_host, int32_t T,
                     void* stream) {
  if (!c || !dout_host || !W_gate_up || !W_down || !dx_host || !dW_gate_up || !dW_down || T <= 0 ||
      T > c->shape.T_max)
    return MOE_ERR_INVALID_ARG;
  if (!c->train() || c->saved_T != T) return MOE_ERR_STATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  c->begin_call(st);
  const moe_shape& s = c->shape;
  const WsPlan& p = c->plan;
  int rc = ensure_copy_streams(c);
  if (rc) return rc;
  // dout has a staging buffer of its own and goes in on the copy-in stream: it arrives while the
  // forward that was enqueued before this call is still computing
  if (c->dout_used) MOE_CUDA(cudaStreamWaitEvent(c->h2d_stream, c->ev_dout_free, 0));
  MOE_CUDA(cudaMemcpyAsync(c->ws + p.st_dout, dout_host, 2 * (size_t)T * s.d, cudaMemcpyHostToDevice, c->h2d_stream));
  MOE_CUDA(cudaEventRecord(c->ev_h2d_done, c->h2d_stream));
  MOE_CUDA(cudaStreamWaitEvent(st, c->ev_h2d_done, 0));
  rc = run_bwd(c, c->at<uint16_t>(p.st_dout), W_gate_up, W_down, c->at<uint16_t>(p.st_dx), dW_gate_up, dW_down,
               d_topk_w_host ? c->at<float>(p.st_dw) : nullptr, T, st, dx_host);
  if (rc) return rc;
  MOE_CUDA(cudaEventRecord(c->ev_dout_free, st));
  c->dout_used = true;
  if (d_topk_w_host)
    MOE_CUDA(cudaMemcpyAsync(d_topk_w_host, c->ws + p.st_dw, sizeof(float) * (size_t)T * s.k,
                             cudaMemcpyDeviceToHost, st));
  return join_out_copy(c, st);   // the forward's deferred result is complete once this call's work on `st` is
}

int moe_get_status(moe_ctx* c, int32_t* code, int32_t* detail) {
  if (!c) return MOE_ERR_INVALID_ARG;
  MOE_CUDA(cudaStreamSynchronize(c->last_stream));
  if (c->out_pending) {
    MOE_CUDA(cudaEventSynchronize(c->ev_out_done));
    c->out_pending = false;
  }
  DevStatus h;
  MOE_CUDA(cudaMemcpy(&h, c->status(), sizeof h, cudaMemcpyDeviceToHost));
  if (code) *code = h.code;
  if (detail) *detail = h.detail;
  if (h.code || h.abort) MOE_CUDA(cudaMemset(c->status(), 0, sizeof h));
  return MOE_OK;
}

int moe_last_launch_count(const moe_ctx* c) { return c ? c->launches : 0; }

int moe_set_wait_budget_ms(moe_ctx* c, int32_t ms) {
  if (!c || ms < 1) return MOE_ERR_INVALID_ARG;
  c->budget_ns = (uint64_t)ms * 1000 * 1000;
  return MOE_OK;
}

int moe_set_profiling(moe_ctx* c, int32_t on) {
  if (!c) return MOE_ERR_INVALID_ARG;
  if (on && !c->events_made) {
    for (int i = 0; i < MOE_NUM_PHASES; ++i) {
      MOE_CUDA(cudaEventCreate(&c->ev_start[i]));
      MOE_CUDA(cudaEventCreate(&c->ev_stop[i]));
    }
    c->events_made = true;
  }
  c->profiling = on != 0;
  return MOE_OK;
}

int moe_get_phase_ms(moe_ctx* c, float* ms) {
  if (!c || !ms) return MOE_ERR_INVALID_ARG;
  for (int i = 0; i < MOE_NUM_PHASES; ++i) {
    ms[i] = 0.f;
    if (c->events_made && c->phase_used[i]) {
      MOE_CUDA(cudaEventSynchronize(c->ev_stop[i]));
      MOE_CUDA(cudaEventElapsedTime(&ms[i], c->ev_start[i], c->ev_stop[i]));
    }
  }
  return MOE_OK;
}

int moe_debug_set_unreachable_dependency(moe_ctx* c, int32_t on) {
  if (!c) return MOE_ERR_INVALID_ARG;
  c->dep_extra = on ? 1 : 0;
  return MOE_OK;
}

int moe_debug_set_plain_launch(moe_ctx* c, int32_t on) {
  if (!c) {   // the context-free scheduling microbenchmark
    study_plain_launch().store(on != 0);
    return MOE_OK;
  }
  c->plain_launch = on != 0;
  return MOE_OK;
}

int moe_debug_buffer(moe_ctx* c, int which, void** ptr, size_t* elems) {
  if (!c || !ptr || !elems) return MOE_ERR_INVALID_ARG;
  const moe_shape& s = c->shape;
  const WsPlan& p = c->plan;
  const size_t Ep = s.E + s.n_shared, slots = (size_t)s.T_max * (s.k + s.n_shared), cap = p.cap_rows;
  const bool train = c->train();
  size_t off = 0, n = 0;
  switch (which) {
    case MOE_BUF_COUNTS: off = p.counts; n = Ep; break;
    case MOE_BUF_OFFSETS: off = p.offsets; n = Ep + 1; break;
    case MOE_BUF_ROW_OF: off = p.row_of; n = slots; break;
    case MOE_BUF_SRC_OF: off = p.src_of; n = slots; break;
    case MOE_BUF_PROW_OF: off = p.prow_of; n = slots; break;
    case MOE_BUF_PAD_OFF: off = p.pad_off; n = Ep + 1; break;
    case MOE_BUF_XP: off = p.Xp; n = cap * s.d; break;
    case MOE_BUF_H: if (!train) return MOE_ERR_STATE; off = p.H; n = cap * 2 * s.F; break;
    case MOE_BUF_A: off = p.A; n = cap * s.F; break;
    case MOE_BUF_Y: off = p.Y; n = cap * s.d; break;
    case MOE_BUF_DOUTP: if (!train) return MOE_ERR_STATE; off = p.dOutp; n = cap * s.d; break;
    case MOE_BUF_DH: if (!train) return MOE_ERR_STATE; off = p.dH; n = cap * 2 * s.F; break;
    case MOE_BUF_DXP: off = p.Y; n = cap * s.d; break;
    case MOE_BUF_META: off = p.meta; n = 8; break;
    case MOE_BUF_TRACE: if (!p.trace_cap) return MOE_ERR_STATE; off = p.trace; n = (size_t)p.trace_cap * 8; break;
    case MOE_BUF_EVENT_COUNTERS: off = p.ctr; n = p.ctr_count; break;
    default: return MOE_ERR_INVALID_ARG;
  }
  *ptr = c->ws + off;
  *elems = n;
  return MOE_OK;
}

// Host-only check of the static schedule (no GPU needed): builds the layout tables and the per-pair
// matrix queues for the given per-expert row counts and lets `pairs` matrix workers (each walking its
// own statically ordered queue) and `vec_workers` vector workers (tickets) run, each blocking on its
// item's dependent counters.
int moe_debug_simulate_schedule(const int32_t* counts, int32_t Ep, int32_t T, int32_t k, int32_t n_shared, int32_t d,
                                int32_t F, int32_t is_bwd, int32_t pairs, int32_t vec_workers, int64_t* stats) {
  if (!counts || Ep < 1 || pairs < 1 || vec_workers < 1 || d < 8 || F < 16) return MOE_ERR_INVALID_ARG;
  // the tables of the layout kernels
  std::vector<int> mb_start(Ep + 1, 0), pair_start(Ep + 1, 0), work_start(Ep + 1, 0);
  for (int e = 0; e < Ep; ++e) {
    const int m = (counts[e] + BLOCK_M - 1) / BLOCK_M, pr = (m + 1) >> 1;
    mb_start[e + 1] = mb_start[e] + m;
    pair_start[e + 1] = pair_start[e] + pr;
    work_start[e + 1] = work_start[e] + pr - (expert_merges(counts[e], m) ? 1 : 0);
  }
  const int M = mb_start[Ep];
  std::vector<int> pblk(pair_start[Ep] + 1, 0), wblk(work_start[Ep] + 1, 0);
  for (int e = 0; e < Ep; ++e) {
    for (int i = pair_start[e]; i < pair_start[e + 1]; ++i) pblk[i] = e;
    for (int i = work_start[e]; i < work_start[e + 1]; ++i) wblk[i] = e;
  }
  ChainParams cp;
  memset(&cp, 0, sizeof cp);
  cp.is_bwd = is_bwd; cp.Ep = Ep; cp.T = T; cp.k = k; cp.kp = k + n_shared; cp.want_dw = 1;
  if (!is_bwd) {
    cp.n_phases = 2; cp.ntn[0] = (F + 127) / 128; cp.ntn[1] = (d + 255) / 256; cp.merges[1] = 1;
  } else {
    cp.n_phases = 4; cp.ntn[0] = (F + 255) / 256; cp.ntn[1] = (F + 255) / 256; cp.strips[1] = (d + 255) / 256;
    cp.ntn[2] = (d + 255) / 256; cp.merges[2] = 1; cp.ntn[3] = (d + 255) / 256; cp.strips[3] = (2 * F + 255) / 256;
  }
  // items of every phase: {first M-block, M-blocks of unit a, M-blocks of unit b} (strips: the expert's M-blocks)
  struct Item { int phase, mb_first, mb_a, mb_b; };
  std::vector<std::vector<Item>> queue(pairs);
  long n_items = 0;
  std::vector<std::vector<int>> cover(cp.n_phases, std::vector<int>(M + 1, 0));
  for (int ph = 0; ph < cp.n_phases; ++ph) {
    if (cp.strips[ph]) {
      const int total = Ep * cp.strips[ph];
      for (int sidx = 0; sidx < total; ++sidx) {
        const int e = sidx / cp.strips[ph];
        queue[sidx % pairs].push_back(Item{ph, mb_start[e], mb_start[e + 1] - mb_start[e], 0});
        ++n_items;
      }
    } else {
      const bool mg = cp.merges[ph] != 0;
      const int total = (mg ? work_start[Ep] : pair_start[Ep]) * cp.ntn[ph];
      const int first = n_shared > 0 ? (mg ? work_start[Ep - n_shared] : pair_start[Ep - n_shared]) * cp.ntn[ph] : 0;
      for (int tq = 0; tq < total; ++tq) {
        const int t = rotate_index(tq, first, total);   // shared experts first (schedule.h)
        const SwapItem it = decode_swap_item(t, cp.ntn[ph], mg, mg ? work_start.data() : pair_start.data(),
                                             mg ? wblk.data() : pblk.data(), mb_start.data());
        if (it.e < 0 || it.e >= Ep || it.nb < 0 || it.nb >= cp.ntn[ph]) return 10;
        if (it.mb_first < mb_start[it.e] || it.mb_first + it.mb_count > mb_start[it.e + 1] || it.mb_count < 1 ||
            it.mb_count > 3 || it.mb_count_a < 1)
          return 10;
        for (int q = 0; q < it.mb_count; ++q) cover[ph][it.mb_first + q]++;
        queue[tq % pairs].push_back(Item{ph, it.mb_first, it.mb_count_a, it.mb_count - it.mb_count_a});
        ++n_items;
      }
    }
  }
  // 1. coverage: every M-block is covered by every column tile of every row-space phase exactly once
  for (int ph = 0; ph < cp.n_phases; ++ph)
    if (!cp.strips[ph])
      for (int mb = 0; mb < M; ++mb)
        if (cover[ph][mb] != cp.ntn[ph]) return 13;
  // 2. execution with a bounded number of workers
  std::vector<long> ctr(ctr_ints(M + 1), 0);
  std::vector<size_t> cursor(pairs, 0);
  const int ngather = gather_total(M), npost = post_total(cp, M);
  struct VecWorker { bool holding = false; VecTask v; };
  std::vector<VecWorker> vw(vec_workers);
  // rows of each token (slot order is irrelevant here): token t's k+S rows live in M-blocks drawn round-robin
  auto token_mblocks_done = [&](int t0, int t1) {
    if (M == 0) return true;
    for (int t = t0; t < t1; ++t)
      for (int j = 0; j < cp.kp; ++j)
        if (ctr[ctr_index((int)(((long)t * cp.kp + j) % M), CTR_DONE)] < thr_done(cp)) return false;
    return true;
  };
  long done_mat = 0, done_vec = 0, rounds = 0, stalls = 0;
  int next_gather = 0, next_post = 0;
  const int vtotal = ngather + npost;
  while (done_mat < n_items || done_vec < vtotal) {
    bool progress = false;
    for (int q = 0; q < pairs; ++q) {
      if (cursor[q] >= queue[q].size()) continue;
      const Item& it = queue[q][cursor[q]];
      const int wk = phase_wait_kind(cp, it.phase), thr = phase_wait_thr(cp, it.phase);
      bool ready = true;
      for (int m = 0; m < it.mb_a + it.mb_b; ++m)
        if (ctr[ctr_index(it.mb_first + m, wk)] < thr) ready = false;
      if (!ready) { ++stalls; continue; }
      const int tk = phase_trigger_kind(cp, it.phase);
      if (tk >= 0)
        for (int m = 0; m < it.mb_a + it.mb_b; ++m) ctr[ctr_index(it.mb_first + m, tk)] += SIG;
      ++cursor[q]; ++done_mat; progress = true;
    }
    for (size_t wi = 0; wi < vw.size(); ++wi) {
      auto& w = vw[wi];
      // worker 0 is a background gatherer; the others leave the gather queue after the first M-blocks
      const bool may_gather = next_gather < ngather && (wi == 0 || next_gather < GATHER_SUB * GATHER_FAST_MBLOCKS);
      if (!w.holding && may_gather) {
        w.v.op = VEC_GATHER; w.v.idx = next_gather++;
        w.holding = true;
        progress = true;
      } else if (!w.holding && next_post < npost && (wi != 0 || next_gather >= ngather)) {
        w.v = decode_post_ticket(cp, next_post++, M);
        w.holding = true;
        progress = true;
      }
      if (!w.holding) continue;
      bool ready = true;
      if (w.v.op == VEC_DW)
        ready = ctr[ctr_index(rotate_index(w.v.idx, n_shared > 0 ? mb_start[Ep - n_shared] : 0, M), CTR_ACTIVATED)] >= thr_activated(cp);
      if (w.v.op == VEC_COMBINE)
        ready = token_mblocks_done(w.v.idx * COMBINE_TOKENS, std::min(T, (w.v.idx + 1) * COMBINE_TOKENS));
      if (!ready) { ++stalls; continue; }
      if (w.v.op == VEC_GATHER)
        ctr[ctr_index(rotate_index(w.v.idx, n_shared > 0 ? mb_start[Ep - n_shared] * GATHER_SUB : 0, ngather) / GATHER_SUB, CTR_GATHERED)] += 1;
      w.holding = false;
      ++done_vec;
      progress = true;
    }
    ++rounds;
    if (!progress) return 20;  // deadlock
  }
  // 3. every counter ends exactly at its threshold
  for (int mb = 0; mb < M; ++mb)
    if (ctr[ctr_index(mb, CTR_GATHERED)] != thr_gathered() || ctr[ctr_index(mb, CTR_ACTIVATED)] != thr_activated(cp) ||
        ctr[ctr_index(mb, CTR_DONE)] != thr_done(cp))
      return 30;
  if (stats) { stats[0] = n_items; stats[1] = vtotal; stats[2] = rounds; stats[3] = stalls; }
  return MOE_OK;
}

int moe_debug_trace(moe_ctx* c, moe_trace_record* records, size_t max_records, size_t* n_written) {
  if (!c || !n_written || (!records && max_records)) return MOE_ERR_INVALID_ARG;
  if (!c->plan.trace_cap) return MOE_ERR_STATE;
  MOE_CUDA(cudaStreamSynchronize(c->last_stream));
  int produced = 0;
  MOE_CUDA(cudaMemcpy(&produced, c->at<int>(c->plan.ctr) + CTR_TRACE_CURSOR, sizeof(int), cudaMemcpyDeviceToHost));
  *n_written = (size_t)produced;
  size_t n = std::min<size_t>(std::min<size_t>((size_t)produced, (size_t)c->plan.trace_cap), max_records);
  if (n == 0) return MOE_OK;
  std::vector<uint32_t> raw(n * 8);
  MOE_CUDA(cudaMemcpy(raw.data(), c->ws + c->plan.trace, n * 32, cudaMemcpyDeviceToHost));
  for (size_t i = 0; i < n; ++i) {
    const uint32_t* r = &raw[8 * i];
    moe_trace_record& o = records[i];
    o.t0_ns = (uint64_t)r[0] | ((uint64_t)r[1] << 32);
    o.t1_ns = (uint64_t)r[2] | ((uint64_t)r[3] << 32);
    o.role = (uint8_t)(r[4] & 0xFF);
    o.phase = (uint8_t)((r[4] >> 8) & 0xFF);
    o.pad = 0;
    o.item = (int32_t)r[5];
    o.cta = r[6];
    o.dep_ns = r[7];
  }
  return MOE_OK;
}

const char* moe_strerror(int code) {
  switch (code) {
    case MOE_OK: return "ok";
    case MOE_ERR_INVALID_ARG: return "invalid argument";
    case MOE_ERR_WORKSPACE: return "workspace too small or misaligned";
    case MOE_ERR_CUDA: return "CUDA call failed";
    case MOE_ERR_NO_DEVICE: return "no sm_100 CUDA device is current";
    case MOE_ERR_STATE: return "no matching saved forward (or context created without MOE_FLAG_SAVE_FOR_BWD)";
    case MOE_ERR_TOO_LARGE: return "size beyond a fixed limit";
    case MOE_ERR_BAD_EXPERT_ID: return "expert id out of range (slot dropped)";
    case MOE_ERR_TIMEOUT: return "bounded device-side wait expired";
    default: return "unknown code";
  }
}

const char* moe_last_cuda_error(void) { return g_cuda_error.c_str(); }

}  // extern "C"
