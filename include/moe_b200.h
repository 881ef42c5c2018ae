/*
 * moe_b200 -- Dispatch->Combine MoE-FFN layer for NVIDIA B200 (sm_100a), C ABI.
 *
 * The layer is the one the paper schedules as a tile-level taskflow (Section 2.2):
 * forward  = Dispatch, GroupedGEMM (gate+up), SwiGLU, GroupedGEMM (down), Combine;
 * backward = backward Dispatch, GMM act_grad, GMM w2_grad, SwiGLU_grad, GMM gate_grad,
 *            GMM w1_grad, backward Combine.
 * On one GPU Dispatch and Combine are local permutes.  Every step runs in hand-written
 * CUDA kernels of this library; there is no CPU fallback.
 *
 * Conventions
 *   - Unless a parameter says "host", every tensor pointer is a DEVICE pointer owned by the
 *     caller, row-major, 16-byte aligned.  The library neither frees nor keeps it after the
 *     call's work has finished on `stream`.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls
 *     only enqueue work; they do not synchronise unless stated.
 *   - bf16 tensors are passed as uint16_t (raw bits).
 *   - Shapes: T tokens, d hidden, E routed experts, k routed experts per token, S shared
 *     experts (taken by every token with weight 1), F expert intermediate size.
 *     Requirements: d % 8 == 0, F % 8 == 0, 1 <= k <= E <= 1024, T <= T_max.
 *   - Weights: W_gate_up[E+S][2F][d] (rows 0..F-1 = gate projection, F..2F-1 = up projection,
 *     d contiguous) and W_down[E+S][d][F] (F contiguous); shared experts are the last S slabs.
 *   - Return value: 0 on success; a negative MOE_ERR_* when an argument is rejected (nothing
 *     was enqueued).  Conditions found by kernels (an expert id out of range, a bounded wait
 *     that ran out) are recorded in the context and read with moe_get_status(); kernels always
 *     terminate.
 *   - A context serialises nothing: use one context per stream, and do not overlap two calls
 *     on the same context.  Contexts on different GPUs of one process, and host threads with
 *     their own contexts, may call concurrently.
 *   - Launch modes: by default a pass is ONE persistent launch (after the index-only layout
 *     kernels) in which gather, GEMM and combine tiles are ordered by event counters;
 *     MOE_FLAG_SERIAL_LAUNCH runs one launch per operator.  Shapes with F % 16 != 0 always take
 *     the one-launch-per-operator path.
 *   - Test and diagnostic entry points (workspace views, schedule simulation, failure injection,
 *     trace read-out) are declared in moe_b200_debug.h.
 */
#ifndef MOE_B200_H
#define MOE_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct moe_ctx moe_ctx; /* opaque: shape, workspace carving, tensor maps, status word */

typedef struct {
  int32_t T_max;    /* largest token count any call will pass */
  int32_t d;        /* hidden size */
  int32_t E;        /* routed experts */
  int32_t k;        /* routed experts per token */
  int32_t n_shared; /* S */
  int32_t F;        /* expert intermediate size */
  uint32_t flags;   /* MOE_FLAG_* */
} moe_shape;

enum {
  MOE_FLAG_RENORM_TOPK = 1u,   /* moe_route: divide the k scores by their sum */
  MOE_FLAG_SAVE_FOR_BWD = 2u,  /* moe_ffn_fwd keeps layout, gathered x, pre-activations and
                                  activations in the workspace for the next moe_ffn_bwd */
  MOE_FLAG_SERIAL_LAUNCH = 4u, /* run the layer as one kernel launch per operator (the paper's
                                  operator-by-operator baseline, Section 5.2) instead of the
                                  single persistent dependency-driven launch */
  MOE_FLAG_SIGMOID_GATE = 16u, /* routing scores are per-expert sigmoids of the logits instead of a softmax over all
                                  experts (moe_route, moe_router_fwd, moe_router_bwd); selection rule unchanged */
  MOE_FLAG_DEFER_OUT_COPY = 32u, /* moe_ffn_fwd_host only: the copy of `out` to the host runs behind whatever is enqueued
                                    next on the stream (e.g. the backward) instead of in front of it; out_host is complete
                                    once a LATER call on the context -- moe_ffn_bwd_host, the next moe_ffn_fwd_host,
                                    moe_get_status -- has completed, not yet when this call's stream work has */
  MOE_FLAG_TRACE = 8u,         /* the persistent launches record a per-tile trace (role, phase, item,
                                  start and end time) into the workspace; read it with
                                  moe_debug_trace (moe_b200_debug.h).  Costs 8 MB of workspace and one
                                  atomic + two 16-byte stores per tile */
};

enum {
  MOE_OK = 0,
  MOE_ERR_INVALID_ARG = -1,   /* NULL pointer, bad shape, T > T_max, misaligned pointer */
  MOE_ERR_WORKSPACE = -2,     /* caller's workspace too small or misaligned */
  MOE_ERR_CUDA = -3,          /* a CUDA runtime/driver call failed (see moe_last_cuda_error) */
  MOE_ERR_NO_DEVICE = -4,     /* no sm_100 device is current */
  MOE_ERR_STATE = -5,         /* moe_ffn_bwd without a saved forward of the same tensors and T */
  MOE_ERR_TOO_LARGE = -6,     /* size beyond a documented fixed limit */
  /* asynchronous, reported by moe_get_status(): */
  MOE_ERR_BAD_EXPERT_ID = 1,  /* detail = flat slot index of one offending entry */
  MOE_ERR_TIMEOUT = 2,        /* a bounded device-side wait expired; detail = where */
};

/* Bytes of device workspace a context of this shape needs (layout arrays, expert-ordered
 * activations, tile table, dependency counters).  0 if the shape is invalid. */
size_t moe_workspace_bytes(const moe_shape* shape);

/* Create a context.  `workspace` is device memory of at least moe_workspace_bytes() bytes,
 * 256-byte aligned, owned by the caller and kept alive until moe_destroy(); pass NULL to let the
 * library cudaMalloc (and later free) it on the current device.  Host-side planning done here
 * (workspace carving, tensor maps of workspace tensors) is outside the timed Dispatch->Combine
 * interval, like the paper's schedule compilation (Section 5.1). */
int moe_create(moe_ctx** out, const moe_shape* shape, void* workspace, size_t workspace_bytes);
int moe_destroy(moe_ctx* ctx);

/* Router scores -> top-k (Section 2.2, first paragraph).  logits[T][E] fp32.
 * topk_ids[T][k]: the k largest raw logits, ties to the lower expert id, slots in descending
 * logit order.  topk_w[T][k]: softmax over all E of the selected experts, renormalised over
 * the k when MOE_FLAG_RENORM_TOPK is set (with MOE_FLAG_SIGMOID_GATE: w = 1 / (1 + exp(-logit)) of each selected
 * expert, renormalised over the k the same way).  counts[E] (may be NULL): tokens per routed expert. */
int moe_route(moe_ctx* ctx, const float* logits, int32_t T, int32_t* topk_ids, float* topk_w,
              int32_t* counts, void* stream);

/* Dispatch layout only (Section 2.2, Dispatch: the index part -- which expert-ordered row each
 * routed token copy goes to).  Flat slot i = t*(k+S)+j; slots j >= k are the shared experts E..E+S-1.
 * counts[E+S]; offsets[E+S+1] = exclusive scan; row_of[T*(k+S)] = expert-ordered row of each slot
 * (rows of one expert keep slot order; -1 for a slot whose expert id is out of range);
 * src_of[row] = slot.  Any output may be NULL.  moe_ffn_fwd computes the same layout internally. */
int moe_layout(moe_ctx* ctx, const int32_t* topk_ids, int32_t T, int32_t* counts, int32_t* offsets,
               int32_t* row_of, int32_t* src_of, void* stream);

/* Forward layer (Section 2.2, second paragraph): for every token t
 *   out[t] = sum_j w(t,j) * ( silu(x_t Wg_e^T) * (x_t Wu_e^T) ) Wd_e^T ,  e = expert of slot j,
 * j over the k routed slots (weight topk_w) and the S shared experts (weight 1).
 * x, out: bf16 [T][d]; topk_ids int32 [T][k]; topk_w fp32 [T][k].  bf16 inputs, fp32
 * accumulation, bf16 output. */
int moe_ffn_fwd(moe_ctx* ctx, const uint16_t* x, const int32_t* topk_ids, const float* topk_w,
                const uint16_t* W_gate_up, const uint16_t* W_down, uint16_t* out, int32_t T,
                void* stream);

/* Backward layer (Section 2.2, third paragraph).  Needs the preceding moe_ffn_fwd on this context
 * with MOE_FLAG_SAVE_FOR_BWD and the same x, topk_ids, topk_w (the same pointers: the backward works
 * from the gathered inputs and the layout that forward saved), weights and T; otherwise MOE_ERR_STATE.
 * dout bf16 [T][d] -> dx bf16 [T][d], dW_gate_up bf16 [E+S][2F][d], dW_down bf16 [E+S][d][F]
 * (both overwritten; an expert that received no token gets exact zeros), d_topk_w fp32 [T][k]
 * (gradient of the routing weights; may be NULL). */
int moe_ffn_bwd(moe_ctx* ctx, const uint16_t* dout, const uint16_t* x, const int32_t* topk_ids,
                const float* topk_w, const uint16_t* W_gate_up, const uint16_t* W_down, uint16_t* dx,
                uint16_t* dW_gate_up, uint16_t* dW_down, float* d_topk_w, int32_t T, void* stream);

/* The same two calls for callers whose activations live in HOST memory (pinned memory gives
 * asynchronous copies).  x/topk_ids/topk_w/dout are host pointers copied to the device inside the
 * call; out/dx/d_topk_w are host pointers filled from the device; weights and weight gradients
 * stay device pointers (model state is resident).  The call returns after enqueueing; the host
 * output buffers are valid, and the host input buffers may be reused, once `stream` has been
 * synchronised.  The large inputs (x_host, dout_host) travel on a copy-in stream of the context,
 * started when the call is made: they must hold their final values at that moment (they are not
 * ordered behind earlier work on `stream`), and the copy overlaps whatever the context still has
 * running.  topk_ids_host / topk_w_host are copied in stream order, so the buffers a preceding
 * moe_route_host on the same stream fills can be passed on without a synchronisation.  Results leave
 * on a copy-out stream that `stream` joins before the call's work ends (dx_host while the last
 * weight gradient is still being computed). */
int moe_ffn_fwd_host(moe_ctx* ctx, const uint16_t* x_host, const int32_t* topk_ids_host,
                     const float* topk_w_host, const uint16_t* W_gate_up, const uint16_t* W_down,
                     uint16_t* out_host, int32_t T, void* stream);
int moe_ffn_bwd_host(moe_ctx* ctx, const uint16_t* dout_host, const uint16_t* W_gate_up,
                     const uint16_t* W_down, uint16_t* dx_host, uint16_t* dW_gate_up,
                     uint16_t* dW_down, float* d_topk_w_host, int32_t T, void* stream);

/* Synchronises the stream of the context's last call, then reports what kernels recorded:
 * *code = 0 or MOE_ERR_BAD_EXPERT_ID / MOE_ERR_TIMEOUT, *detail = where.  Clears the record. */
int moe_get_status(moe_ctx* ctx, int32_t* code, int32_t* detail);

/* Number of kernels the context's last call launched (for launch accounting). */
int moe_last_launch_count(const moe_ctx* ctx);

/* Budget, in milliseconds, of every bounded device-side wait (default 2000). */
int moe_set_wait_budget_ms(moe_ctx* ctx, int32_t ms);

/* Per-operator device times.  With profiling on, every later call records CUDA events on its
 * stream between the operators it launches (the operators of Section 2.2; a single persistent
 * launch reports one entry).  moe_get_phase_ms synchronises on the last event of the context's
 * last call and fills ms[MOE_NUM_PHASES] with that call's times (0 for operators it did not run). */
enum {
  MOE_PHASE_ROUTE = 0,
  MOE_PHASE_LAYOUT = 1,        /* histogram + scan + permutation (Dispatch, index part) */
  MOE_PHASE_GATHER = 2,        /* Dispatch, data part */
  MOE_PHASE_GEMM_GATE_UP = 3,  /* GMM1 + SwiGLU */
  MOE_PHASE_GEMM_DOWN = 4,     /* GMM2 */
  MOE_PHASE_COMBINE = 5,
  MOE_PHASE_BWD_GATHER = 6,    /* backward Dispatch */
  MOE_PHASE_ACT_GRAD = 7,      /* GMM act_grad + SwiGLU_grad */
  MOE_PHASE_DW_REDUCE = 8,     /* routing-weight gradient */
  MOE_PHASE_WGRAD_DOWN = 9,    /* GMM w2_grad */
  MOE_PHASE_GATE_GRAD = 10,    /* GMM gate_grad */
  MOE_PHASE_WGRAD_GATE_UP = 11,/* GMM w1_grad */
  MOE_PHASE_BWD_COMBINE = 12,
  MOE_PHASE_FUSED_FWD = 13,    /* the single persistent forward launch */
  MOE_PHASE_FUSED_BWD = 14,    /* the single persistent backward launch */
  MOE_NUM_PHASES = 15,
};
int moe_set_profiling(moe_ctx* ctx, int32_t on);
int moe_get_phase_ms(moe_ctx* ctx, float* ms);

/* moe_route for host buffers: logits_host[T][E] is copied in, topk_ids_host / topk_w_host are
 * filled from the device (valid once `stream` has been synchronised). */
int moe_route_host(moe_ctx* ctx, const float* logits_host, int32_t T, int32_t* topk_ids_host,
                   float* topk_w_host, void* stream);

/* Dispatch layout for callers that cannot allocate device memory (no counterpart in the paper:
 * this is a convenience of this library).  Who needs it: code that runs where cudaMalloc is not
 * allowed or not wanted -- inside a framework's pre-planned memory region, a latency-critical
 * serving loop (cudaMalloc synchronises the device), a plugin that only receives its input and
 * output buffers -- and callers without a moe_ctx.  It computes exactly what moe_layout computes
 * and needs no context: the scratch memory of the layout kernels is a fixed array inside the
 * library (about 1.6 MB held on every GPU that loads the library, until the process exits), and
 * the call performs no cudaMalloc/cudaFree and calls no allocating routine.
 *   topk_ids[T][k] -> counts[E+S], offsets[E+S+1], row_of[T*(k+S)], src_of[T*(k+S)] (all device
 *   pointers, all required); status2 (device int32[2], may be NULL) receives {code, detail}:
 *   {0,0} or {MOE_ERR_BAD_EXPERT_ID, slot}.
 * Limits: T*(k+S) <= MOE_NOALLOC_MAX_SLOTS, E+S <= MOE_NOALLOC_MAX_EXPERTS, and
 * ceil(T*(k+S)/2048)*(E+S) <= 131072; larger problems return MOE_ERR_TOO_LARGE (use moe_layout).
 * The first call on each device looks up the array's device address (with that device current);
 * make that first call outside any stream capture.  All calls share the one array, which keeps the
 * previous call's contents (the call clears what must start at zero): two calls whose work overlaps
 * on the GPU -- different streams, or different threads -- race; serialise them. */
#define MOE_NOALLOC_MAX_SLOTS 262144
#define MOE_NOALLOC_MAX_EXPERTS 1088
int moe_layout_noalloc(const int32_t* topk_ids, int32_t T, int32_t E, int32_t k, int32_t n_shared,
                       int32_t* counts, int32_t* offsets, int32_t* row_of, int32_t* src_of,
                       int32_t* status2, void* stream);

/* ---- Router in the path (Section 2.2, first paragraph: the router assigns each token its top-k experts and
 * their routing scores) -----------------------------------------------------------------------------------
 * moe_router_fwd: logits = x W_r^T on the tensor cores (bf16 operands, fp32 accumulation) with moe_route's
 * softmax top-k fused into the same launch -- same selection rule (raw logits compared, equal logits to the
 * lower expert id, slots in descending order), same scores (softmax over all E, renormalised over the k
 * selected with MOE_FLAG_RENORM_TOPK).
 *   x[T][d] bf16, W_r[E][d] bf16 (router weights, one row per routed expert), both device pointers, 16-byte
 *   aligned -> topk_ids[T][k] int32, topk_w[T][k] fp32; logits[T][E] fp32 (may be NULL: not stored; keep them
 *   for moe_router_bwd), counts[E] int32 (may be NULL).
 * Limits: E <= 256, k <= 8 (MOE_ERR_TOO_LARGE otherwise: compute the logits elsewhere and call moe_route).
 * The logits are fp32 sums in the tensor cores' order: an expert whose logit differs from the k-th largest by
 * less than the rounding of that sum may be selected differently than by an exact computation.
 *
 * moe_router_bwd: gradient of the k scores with respect to the logits (the selection passes none), from
 * d_topk_w[T][k] as moe_ffn_bwd returns it: p = softmax(logits) over all E,
 *   without renormalisation  d_logits[t][e] = [e = e_j] g_j p_e - p_e * sum_j g_j p_{e_j}
 *   with renormalisation     d_logits[t][e_j] = w_j (g_j - sum_i g_i w_i), 0 for experts not selected.
 *   logits[T][E] fp32, topk_ids[T][k], d_topk_w[T][k] fp32 -> d_logits[T][E] fp32 (all device pointers).
 * With MOE_FLAG_SIGMOID_GATE (s = sigmoid of the logit, Z = sum of the selected s): without renormalisation
 * d_logits[t][e_j] = g_j s_j (1 - s_j); with it d_logits[t][e_j] = s_j (1 - s_j) / Z * (g_j - sum_i g_i w_i); 0 elsewhere.
 * The two dense products that follow (d_logits^T x for the router weights, d_logits W_r for x) are plain
 * GEMMs outside this library.  Limit: k <= 32.  Both calls are asynchronous on `stream`. */
int moe_router_fwd(moe_ctx* ctx, const uint16_t* x, const uint16_t* W_r, int32_t T, int32_t* topk_ids,
                   float* topk_w, float* logits, int32_t* counts, void* stream);
int moe_router_bwd(moe_ctx* ctx, const float* logits, const int32_t* topk_ids, const float* d_topk_w, int32_t T,
                   float* d_logits, void* stream);

/* ---- Scheduling microbenchmark: SwiGLU + Add operator pair (Section 6.1, Section 6.2) -------------
 * The two element-wise operators the paper uses to study scheduling in isolation, on
 *   x[M][2C] bf16 (gate | up halves of each row), r[M][C] bf16  ->
 *   s[M][C] = bf16(silu(gate) * up)   (the intermediate, stored in global memory in every mode)
 *   z[M][C] = bf16(s + r)
 * with rows split into tiles of tile_rows, one task per operator and tile, run in one of three ways:
 *   MOE_STUDY_SERIAL   two launches, one per operator (all of SwiGLU, then all of Add);
 *   MOE_STUDY_STATIC   one persistent launch; each worker runs a fixed alternating list of SwiGLU and Add
 *                      tasks, an Add task waiting on the event counter its producer (another worker) raises;
 *   MOE_STUDY_DYNAMIC  one persistent launch; the same tasks and events, dispatched at run time: SwiGLU tasks
 *                      from a ticket, Add tasks from a FIFO ready queue in global memory (a finished SwiGLU
 *                      task appends its Add task; a free worker pops the queue before taking a ticket).
 * All pointers are device pointers, 16-byte aligned; C % 8 == 0; M >= 0 (M == 0 launches nothing and
 * ignores x, r, s and z).
 * workspace: moe_sched_study_workspace_bytes(M, tile_rows) bytes of device memory owned by the caller, cleared
 * by the call; it holds the status word, the queue and the event counters, and afterwards the workers'
 * dispatch accounting, which moe_sched_study_stats() reads back (it synchronises the stream):
 *   status2[2] = {code, detail} ({0,0}, or MOE_ERR_TIMEOUT and the tile whose wait ran out after 2 s),
 *   dispatch_ns = summed over workers, the time between the end of one task's work and the start of the
 *   next one's (ticket, decode, queue and event waits); tasks = the number of tasks that ran (2 * tiles;
 *   both are 0 in the serial mode).  Any of the three may be NULL.
 * Returns MOE_OK or MOE_ERR_INVALID_ARG / MOE_ERR_WORKSPACE / MOE_ERR_NO_DEVICE / MOE_ERR_CUDA. */
#define MOE_STUDY_SERIAL 0
#define MOE_STUDY_STATIC 1
#define MOE_STUDY_DYNAMIC 2
size_t moe_sched_study_workspace_bytes(int32_t M, int32_t tile_rows);
int moe_sched_study(int32_t mode, const uint16_t* x, const uint16_t* r, uint16_t* s, uint16_t* z,
                    int32_t M, int32_t C, int32_t tile_rows, void* workspace, size_t workspace_bytes,
                    void* stream);
int moe_sched_study_stats(const void* workspace, int32_t* status2, uint64_t* dispatch_ns,
                          uint64_t* tasks, void* stream);

/* ---- Generic taskflow front end (Section 4.2: Operator Dependency Graph, SplitSpec, Algorithm 1 "Split
 * Propagation", Table 1 Task Descriptor; Section 4.3: queues, events with static thresholds) ---------------
 * Host side: an operator graph over 2-D bf16 tensors is compiled into Task Descriptors (TDs) and one statically
 * ordered vector queue; device side: a persistent runtime whose workers take the next TD of the queue, wait for
 * its dependent event, run the handler named by task_type on the TD's row range, and raise its trigger event.
 * The runtime knows handlers, not graphs: any chain of the operators below runs without new device code.
 *
 * Tensors: moe_tf_tensor {rows, cols}, row-major bf16; tensor ids are indices into the array.  A tensor no
 * operator produces is an input of the graph.
 * Operators (moe_tf_operator): op = MOE_TF_SWIGLU (inputs {x[M][2C]} -> outputs {s[M][C]}) or MOE_TF_ADD
 * (inputs {a, b}[M][C] -> {z[M][C]}); SplitSpec fields as in Section 4.2:
 *   n_split_inputs = -1: the operator is a partition origin (split_inputs = None); otherwise it splits only
 *     if input split_input_idx[i] carries the label split_input_dim[i] for every i (inputs not listed are
 *     ignored by the check, like the metadata inputs of Combine), else it falls back to ONE unsplit task;
 *   split_output_dim[j]: the label written on output j when the operator is split (-1: none);
 *   task_rows: task_num_fn = ceil(rows of output 0 / task_rows).  Only dimension 0 (rows) can be split.
 * moe_taskflow_compile (host only, no GPU needed) runs Algorithm 1, fills the TDs (Table 1's fields; TDesc =
 * {tensor slot, row offset, rows, cols}), assigns events -- one counter per row block of a group of tensors
 * that are consumed together, threshold = the number of TDs that write into the block -- and orders the queue:
 * a topological order that runs a consumer task `lag_rows` rows behind its producers, so that intermediates are
 * read back while still in L2 (Section 4.5).  Outputs: tds[0..*n_tds) in queue order, *n_events,
 * op_task_num[n_ops] (Algorithm 1's task_num), tensor_split_dim / tensor_split_num [n_tensors] (its labels).
 * Task granularities that feed one event must be multiples of one another, and an operator may not consume a
 * tensor of the event group it triggers: MOE_ERR_INVALID_ARG.  td_cap too small: MOE_ERR_WORKSPACE.
 *
 * moe_taskflow_run: tds (host), slots[n_tensors] (host array of DEVICE pointers, 16-byte aligned, cols % 8 == 0),
 * workspace (device, moe_taskflow_workspace_bytes; its counters are cleared by every call) -> launches the runtime
 * on `stream`.  upload != 0 copies the descriptor table and the slot table into the workspace first; upload == 0
 * reuses what an earlier call with the same tds, slots and workspace put there (a compiled plan is uploaded once
 * and run every step; tds and slots are still checked on the host either way, and a run whose workspace does not
 * hold this plan -- judged by its sizes, its slot pointers and its first and last descriptor -- does nothing and reports
 * {MOE_ERR_BAD_EXPERT_ID, n_tds} through moe_taskflow_status).
 * moe_taskflow_status (synchronises the stream): status2 = {code, detail} ({0,0} or MOE_ERR_TIMEOUT and the TD
 * whose wait ran out after 2 s). */
#define MOE_TF_SWIGLU 1
#define MOE_TF_ADD 2
#define MOE_TF_QUEUE_MATRIX 0
#define MOE_TF_QUEUE_VECTOR 1
#define MOE_TF_NO_EVENT 0xFFFFFFFFu
typedef struct { int32_t rows, cols; } moe_tf_tensor;
typedef struct {
  int32_t op;
  int32_t n_inputs, inputs[4];
  int32_t n_outputs, outputs[2];
  int32_t n_split_inputs, split_input_idx[4], split_input_dim[4];
  int32_t split_output_dim[2];
  int32_t task_rows;
} moe_tf_operator;
typedef struct { uint32_t slot, row_offset, rows, cols; } moe_tf_tdesc;
typedef struct {
  uint32_t task_type, queue_type;
  uint32_t dependent_event, dependent_threshold, trigger_event;
  uint32_t task_index, task_split_num, task_split_value;   /* tile index, tiles of the operator, rows per tile */
  uint32_t tiling_data_position;                           /* index of the operator in the graph */
  uint32_t n_inputs, n_outputs;
  moe_tf_tdesc inputs[4], outputs[2];
} moe_tf_td;
int moe_taskflow_compile(const moe_tf_tensor* tensors, int32_t n_tensors, const moe_tf_operator* ops, int32_t n_ops,
                         int32_t lag_rows, moe_tf_td* tds, int32_t td_cap, int32_t* n_tds, int32_t* n_events,
                         int32_t* op_task_num, int32_t* tensor_split_dim, int32_t* tensor_split_num);
size_t moe_taskflow_workspace_bytes(int32_t n_tds, int32_t n_events, int32_t n_tensors);
int moe_taskflow_run(const moe_tf_td* tds, int32_t n_tds, int32_t n_events, void* const* slots, int32_t n_tensors,
                     void* workspace, size_t workspace_bytes, int32_t upload, void* stream);
int moe_taskflow_status(const void* workspace, int32_t* status2, void* stream);

/* ---- Expert parallelism over peer memory: one-sided put + signal (Section 4.1 put_mem_signal and the
 * taskization of the Dispatch / Combine AllToAll; Section 4.5 rank-aware task reordering) --------------------
 * R ranks, expert e on rank e / (E / R).  Every rank exposes a moe_ep_peer: buffers in ITS memory that the other
 * ranks write into with plain peer stores, each followed by a release-increment of a counter beside the buffer;
 * the owner's consumers poll those counters locally.  No collective, no multicast load, no remote load.
 *   recv[recv_rows][d] bf16: the rows of the rank's experts ordered by (expert, source rank, source slot t*k+j);
 *   recv_meta[recv_rows][4] int32: source rank, source slot, routing weight (fp32 bits), 0;
 *   recv_counters[ceil(recv_rows / MOE_EP_BLOCK_ROWS)]: rows that have arrived in each block of the receive buffer
 *     (its threshold: the rows the block holds);
 *   ret[T * k][d] bf16: expert outputs returned to the token's rank, indexed by slot;
 *   ret_counters[ceil(T / MOE_EP_TOKEN_BLOCK)]: rows returned per block of tokens (threshold: tokens * k).
 * All pointers in a moe_ep_peer must be valid device addresses ON THE CALLING DEVICE (peer mappings for remote
 * ranks), 16-byte aligned; d % 8 == 0.
 *
 * moe_ep_plan (host only): from the all-gathered per-rank expert counts[R][E] it gives rank `rank` its list of
 * communication tasks -- tiles of up to MOE_EP_TILE_ROWS rows of one expert: {expert, first local expert-ordered
 * row, rows, destination rank, first destination row} -- in rank-rotated order (destinations rank+1, rank+2, ...,
 * rank itself last), the rows every rank receives, and the first receive row of each of `rank`'s own experts.
 *
 * moe_ep_dispatch: for every rank in locals[] (one per process in a real deployment; all R in a single-GPU
 * emulation, where one cooperative launch plays every rank) producer blocks take tasks by ticket, gather the
 * task's rows of x (through src_of from moe_layout over all E experts, n_shared = 0) into the destination's recv
 * and recv_meta, and signal the destination's recv_counters; consumer blocks of the same launch wait for each
 * block's counter and copy the block into `consumed` (if not NULL) -- the stand-in for the grouped-GEMM tiles
 * that would start on the block.  moe_ep_combine: producer blocks return each row of y (expert outputs in
 * receive order) to ret[slot] of its source rank and signal ret_counters; consumer blocks wait per token block
 * and write out[t] = sum_j ret[t*k+j] (fp32, slot order).
 * The calls clear the counters, tickets and status of the ranks in locals[]: with more than one process the
 * caller must place a barrier between two calls so that no rank signals a counter before its owner cleared it.
 * status (device int32[4], cleared by the call): {code, detail, ..} = MOE_ERR_TIMEOUT if a bounded wait ran out.
 * Returns MOE_OK / MOE_ERR_INVALID_ARG / MOE_ERR_WORKSPACE (task_cap) / MOE_ERR_NO_DEVICE / MOE_ERR_CUDA. */
#define MOE_EP_MAX_RANKS 8
#define MOE_EP_TILE_ROWS 32
#define MOE_EP_BLOCK_ROWS 128
#define MOE_EP_TOKEN_BLOCK 32
typedef struct {
  uint16_t* recv;
  int32_t* recv_meta;
  int32_t* recv_counters;
  uint16_t* ret;
  int32_t* ret_counters;
} moe_ep_peer;
typedef struct { int32_t expert, src_row0, nrows, dst_rank, dst_row0; } moe_ep_task;
typedef struct {
  int32_t rank, T, n_tasks, recv_rows;
  const uint16_t* x;          /* [T][d] */
  const float* topk_w;        /* [T][k] */
  const int32_t* src_of;      /* [T*k] */
  const moe_ep_task* tasks;   /* device copy of the plan's task list */
  uint16_t* consumed;         /* [recv_rows][d] or NULL */
  int32_t* ticket;            /* device int32[2]: task tickets of this rank */
} moe_ep_local;
typedef struct {
  int32_t rank, T, recv_rows, pad;
  const uint16_t* y;          /* [recv_rows][d] */
  uint16_t* out;              /* [T][d] */
  int32_t* ticket;            /* device int32[2] */
} moe_ep_local_combine;
int moe_ep_plan(const int32_t* counts, int32_t R, int32_t E, int32_t rank, moe_ep_task* tasks, int32_t task_cap,
                int32_t* n_tasks, int32_t* recv_rows, int32_t* recv_expert_offsets);
int moe_ep_dispatch(const moe_ep_peer* peers, const moe_ep_local* locals, int32_t n_local, int32_t R, int32_t k,
                    int32_t d, int32_t* status, void* stream);
int moe_ep_combine(const moe_ep_peer* peers, const moe_ep_local_combine* locals, int32_t n_local, int32_t R,
                   int32_t k, int32_t d, int32_t* status, void* stream);

const char* moe_strerror(int code);
/* Text of the last CUDA error a call on this thread ran into ("" if none). */
const char* moe_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* MOE_B200_H */
