// Warp roles of the CTA-pair grouped GEMMs as device functions: TMA producers, tcgen05.mma issuer and
// epilogue warps of the token-column row-space operators and of the strip-wise weight gradients.
//
// Every function here handles ONE work item (a token tile x column tile of a row-space operator, or a
// strip of a weight gradient), already decoded, for one role: decoding an item takes a chain of dependent
// global loads (two or three microseconds), so callers decode the NEXT item while the current one runs.  The one-launch-per-operator kernels (gemm_tc3.cu,
// gemm_wgrad.cu) walk an operator's items in a static order with no event counters; the persistent
// launch (fused.cu) takes items of all operators of a pass from one ticket queue, carries the pipeline
// state (stage ring position, barrier parities, accumulator parity) from item to item and orders
// tiles by event counters (the dependent and trigger events of Section 4.3).  Both use exactly this
// code, so they produce the same bits.
#pragma once

#include "gemm_swap.cuh"

namespace moe {

constexpr int PIPE_STAGES = 5;   // row-space operators: operand stages of 16 KB of weights + 16..24 KB of tokens;
                                 // weight gradients: 16 KB slots of the strip's A operand
constexpr int WG_B_STAGES = 7;   // weight gradients: 16 KB stages of the streamed B operand
constexpr int MAX_STAGES = 8;

struct __align__(8) PipeBarriers {
  uint64_t full[MAX_STAGES];      // used in the even CTA: bytes of both CTAs' loads of the stage
  uint64_t empty[MAX_STAGES];     // in each CTA: the stage's MMAs are complete
  uint64_t a_empty[PIPE_STAGES];  // weight gradients, in each CTA: every MMA that reads the A slot's content is complete
  uint64_t tmem_full[2];          // in each CTA: accumulator ready
  uint64_t tmem_empty[2];         // used in the even CTA: the 8 epilogue warps of the pair have drained it
  uint64_t drain;
  uint32_t tmem_base;
  int epi_phase[EPI_WARPS];       // in each CTA: the phase each epilogue warp is in (its stores of earlier phases have read shared memory)
  int pad;
};

// Pipeline state of a role, carried from item to item (the barriers persist).  The parity to wait for is kept per
// stage, so operators with rings of different depth can follow one another in one launch (the ring position
// restarts at 0 at such a boundary, where every stage has been consumed).
struct LoaderState { uint32_t s = 0, empty_par = (1u << MAX_STAGES) - 1, a_s = 0, a_ph = (1u << PIPE_STAGES) - 1; };
struct IssuerState { uint32_t s = 0, full_par = 0, a_s = 0, acc_it = 0; };
struct EpiState { uint32_t acc_it = 0, round = 0; };   // round: position in the warp's ring of staging slots

__device__ __forceinline__ void pipe_init(PipeBarriers* bars) {   // one thread
  for (int s = 0; s < MAX_STAGES; ++s) {
    mbar_init(&bars->full[s], 1);
    mbar_init(&bars->empty[s], 1);
  }
  for (int s = 0; s < PIPE_STAGES; ++s) mbar_init(&bars->a_empty[s], 1);
  for (int s = 0; s < 2; ++s) {
    mbar_init(&bars->tmem_full[s], 1);
    mbar_init(&bars->tmem_empty[s], 2 * EPI_WARPS);
  }
  mbar_init(&bars->drain, 1);
  for (int w = 0; w < EPI_WARPS; ++w) bars->epi_phase[w] = 0;
}
// Phase boundaries of the persistent launch.  The shared memory of a phase (operand ring, staging) is carved
// per operator, so the roles that write it -- loaders, and epilogue warps (staging) -- enter phase p only when
// every epilogue warp of their CTA has: all MMAs of earlier phases are then complete and every store has read
// its staging slot.  A word per warp rather than an mbarrier: a pair may pass several phases at once.
__device__ __forceinline__ void epi_enter_phase(PipeBarriers* bars, int quad, int phase) {   // one lane
  __threadfence_block();
  *reinterpret_cast<volatile int*>(&bars->epi_phase[quad]) = phase;
}
__device__ __forceinline__ bool phase_wait(PipeBarriers* bars, int phase, const WaitCtl& wc) {   // one lane
  volatile int* c = bars->epi_phase;
  uint64_t t0 = 0;
  for (uint32_t spin = 1; c[0] < phase || c[1] < phase || c[2] < phase || c[3] < phase; ++spin) {
    __nanosleep(100);
    if ((spin & 63u) == 0) {
      if (*reinterpret_cast<volatile int*>(&wc.status->abort)) return false;
      const uint64_t now = globaltimer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > wc.budget_ns) {
        report(wc.status, /*MOE_ERR_TIMEOUT*/ 2, (SITE_EMPTY << 24) | 0xFFFF00 | (phase & 0xFF));
        return false;
      }
    }
  }
  __threadfence_block();
  return true;
}

// After a failed or aborted launch: let the tensor core finish what was issued before TMEM is freed.
__device__ __forceinline__ void issuer_drain(PipeBarriers* bars, DevStatus* status) {   // one lane
  tc_commit_pair(&bars->drain);
  const WaitCtl shortwc{status, 20ull * 1000 * 1000};
  mbar_wait(&bars->drain, 0, shortwc, SITE_DRAIN, 0);
}

// ---------------------------------------------------------------- per-tile trace (optional)
// One 32-byte record per traced interval: {t0, t1} in globaltimer ns, {role | phase << 8, item, CTA,
// ns from t0 until the dependencies were met}.
struct TraceCtl {
  uint4* buf;     // NULL: tracing off
  int cap;        // records
  int* cursor;
};
enum TraceRole : int { TR_SCHED = 0, TR_MMA = 1, TR_EPI = 2, TR_VEC = 3 };
__device__ __forceinline__ void trace_put(const TraceCtl& tr, int role, int phase, int item, uint64_t t0, uint64_t t_dep,
                                          uint64_t t1) {
  const int i = atomicAdd(tr.cursor, 1);
  if (i >= tr.cap) return;   // the cursor keeps counting: the host sees how many records were dropped
  tr.buf[2 * i] = make_uint4((uint32_t)t0, (uint32_t)(t0 >> 32), (uint32_t)t1, (uint32_t)(t1 >> 32));
  tr.buf[2 * i + 1] = make_uint4((uint32_t)(role | (phase << 8)), (uint32_t)item, blockIdx.x, (uint32_t)(t_dep - t0));
}

// ---------------------------------------------------------------- event policies
// No events: the one-launch-per-operator kernels (the kernel boundary orders the operators).
struct NoDeps {
  static constexpr bool kOn = false;
  __device__ __forceinline__ bool wait(int, int, int, int) const { return true; }
  __device__ __forceinline__ void signal(int, int) const {}
  __device__ __forceinline__ bool tracing() const { return false; }
  __device__ __forceinline__ void trace(int, int, uint64_t, uint64_t, uint64_t) const {}
};
// Event counters per M-block with static thresholds.
struct ChainDeps {
  static constexpr bool kOn = true;
  int* ctr;
  int wait_kind, wait_thr;   // dependent event of the phase's items
  int trig_kind;             // trigger event (CTR_NONE: nothing consumes the phase's output inside the launch)
  int phase;
  WaitCtl wc;
  TraceCtl tr;
  // All lanes of a warp: wait until the counters of M-blocks [first, first + count) reach the threshold.
  __device__ __forceinline__ bool wait(int first, int count, int lane, int item) const {
    int ok = 1;
    for (int q = lane; q < count; q += 32)
      if (!counter_wait(ctr + ctr_index(first + q, wait_kind), wait_thr, wc, item)) ok = 0;
    return __all_sync(0xffffffffu, ok) != 0;
  }
  // One lane, after its warp's stores of the tile are complete and ordered (see the epilogue roles).
  __device__ __forceinline__ void signal(int first, int count) const {
    if (trig_kind < 0) return;
    for (int q = 0; q < count; ++q) counter_signal(ctr + ctr_index(first + q, trig_kind), 1);
  }
  __device__ __forceinline__ bool tracing() const { return tr.buf != nullptr; }
  __device__ __forceinline__ void trace(int role, int item, uint64_t t0, uint64_t t_dep, uint64_t t1) const {
    trace_put(tr, role, phase, item, t0, t_dep, t1);
  }
};

// =====================================================================================================
// Token-column row-space operators (gemm_swap.cuh)
// =====================================================================================================
template <int MODE>
__host__ __device__ constexpr int swap_staging_slot_bytes() { return swap_merges<MODE>() ? SW_SLOT_BYTES / 2 : SW_SLOT_BYTES; }
// shared memory of a phase, from the 1024-byte aligned base: weights | tokens | staging | act_grad scratch
template <int MODE>
__host__ __device__ constexpr size_t swap_layout_bytes() {
  return (size_t)PIPE_STAGES * (W_STAGE_BYTES + tok_stage_bytes<MODE>()) + 4 * SW_SLOTS * swap_staging_slot_bytes<MODE>() +
         (MODE == GEMM_ACT_GRAD ? 4 * SW_SCRATCH_BYTES : 0);
}

// TMA producers (both CTAs) of item t.  tok_warp = false: the weights and the stage's byte count; true: the
// tokens.
template <int MODE, class DEP>
__device__ __forceinline__ bool swap_load_item(const GemmArgs& a, uint8_t* smem, PipeBarriers* bars, LoaderState& ls,
                                               bool tok_warp, int rank, int lane, const SwapWork& wk, int t,
                                               const WaitCtl& wc, const DEP& dep) {
  constexpr int TOKB = tok_stage_bytes<MODE>();
  uint8_t* sW = smem;                                    // [PIPE_STAGES][16 KB] weights
  uint8_t* sT = smem + PIPE_STAGES * W_STAGE_BYTES;      // [PIPE_STAGES][TOKB] tokens (this CTA's half)
  // with events: the item was published only after its dependent events were met (acquired by the scheduler,
  // handed on through the ticket ring); what the producers wrote must be seen by the TMA loads
  if (DEP::kOn && tok_warp) fence_proxy_async();
  for (int kb = 0; kb < wk.a.nkb; ++kb) {
    int go = 1;
    if (lane == 0) go = mbar_wait(&bars->empty[ls.s], (ls.empty_par >> ls.s) & 1, wc, SITE_EMPTY, t, 50) ? 1 : 0;
    go = __shfl_sync(0xffffffffu, go, 0);
    if (!go) return false;
    ls.empty_par ^= 1u << ls.s;
    if (!tok_warp) {
      load_weights_swap<MODE>(a, wk.a, kb, rank, sW + ls.s * W_STAGE_BYTES, &bars->full[ls.s], lane, wk.a.ntok + wk.b.ntok);
    } else {
      load_tokens_swap(a, wk.a, kb, rank, sT + ls.s * TOKB, &bars->full[ls.s], lane);
      if (wk.merged)   // lane 1: the second token tile, behind the first in the stage
        load_tokens_swap(a, wk.b, kb, rank, sT + ls.s * TOKB + (wk.a.ntok >> 1) * (BK * 2), &bars->full[ls.s], lane - 1);
    }
    if (++ls.s == PIPE_STAGES) ls.s = 0;
  }
  return true;
}

// MMA issuer: warp 1 of the even CTA.  The whole warp walks the loop (uniform control flow: lanes parked at a
// warp barrier while one lane loops would share that lane's issue slots) and lane 0 (`issue`) alone issues
// the MMAs and commits.  The loop bounds the tensor pipe when a k-block's MMAs are short: stage index, phase
// and descriptor words are carried in registers.
template <int MODE, class DEP>
__device__ __forceinline__ bool swap_issue_item(const GemmArgs& a, uint8_t* smem, PipeBarriers* bars, uint32_t tmem_base,
                                                IssuerState& is, bool issue, const SwapWork& wk, int t,
                                                const WaitCtl& wc, const DEP& dep) {
  constexpr int TOKB = tok_stage_bytes<MODE>();
  const uint32_t w_lo0 = swap_w_desc_lo<MODE>(smem_u32(smem));
  const uint32_t t_lo0 = smem_desc_lo(smem_u32(smem + PIPE_STAGES * W_STAGE_BYTES), 16);
  uint32_t w_lo = w_lo0 + is.s * (W_STAGE_BYTES >> 4), t_lo = t_lo0 + is.s * (TOKB >> 4);
  const int as = is.acc_it & 1;
  if (!mbar_wait(&bars->tmem_empty[as], ((is.acc_it >> 1) & 1) ^ 1, wc, SITE_TMEM_EMPTY, t)) return false;
  if (wk.merged &&   // the second token tile accumulates in the other buffer
      !mbar_wait(&bars->tmem_empty[as ^ 1], (((is.acc_it + 1) >> 1) & 1) ^ 1, wc, SITE_TMEM_EMPTY, t)) return false;
  tc_fence_after_sync();
  const uint32_t d_tmem = tmem_base + as * BN, d_tmem_b = tmem_base + (as ^ 1) * BN;
  const uint32_t idesc = swap_idesc<MODE>(wk.a.ntok), idesc_b = swap_idesc<MODE>(wk.merged ? wk.b.ntok : TOK_GRAIN);
  const uint32_t t_off_b = (uint32_t)((wk.a.ntok >> 1) * (BK * 2)) >> 4;
  uint64_t t0 = 0;
  for (int kb = 0; kb < wk.a.nkb; ++kb) {
    if (!mbar_wait(&bars->full[is.s], (is.full_par >> is.s) & 1, wc, SITE_FULL, t)) return false;
    is.full_par ^= 1u << is.s;
    if (DEP::kOn && kb == 0 && issue && dep.tracing()) t0 = globaltimer_ns();
    tc_fence_after_sync();
    if (issue) {
      mma_kblock_swap<MODE>(d_tmem, w_lo, t_lo, idesc, kb == 0);
      if (wk.merged) mma_kblock_swap<MODE>(d_tmem_b, w_lo, t_lo + t_off_b, idesc_b, kb == 0);
      tc_commit_pair(&bars->empty[is.s]);   // frees the stage in both CTAs
    }
    if (++is.s == PIPE_STAGES) {
      is.s = 0; w_lo = w_lo0; t_lo = t_lo0;
    } else {
      w_lo += W_STAGE_BYTES >> 4; t_lo += TOKB >> 4;
    }
  }
  if (issue) tc_commit_pair(&bars->tmem_full[as]);  // accumulator slices ready in both CTAs
  ++is.acc_it;
  if (wk.merged) {
    if (issue) tc_commit_pair(&bars->tmem_full[as ^ 1]);
    ++is.acc_it;
  }
  if (DEP::kOn && issue && dep.tracing()) dep.trace(TR_MMA, t, t0, t0, globaltimer_ns());
  return true;
}

// Epilogue warps (both CTAs, own features).  With events: a warp signals the M-blocks of a tile once its
// TMA stores of that tile are complete (cp.async.bulk.wait_group 0), ordered for consumers that read
// through TMA (fence.proxy.async) and released at GPU scope.
template <int MODE, class DEP>
__device__ __forceinline__ bool swap_epilogue_item(const GemmArgs& a, uint8_t* smem, PipeBarriers* bars,
                                                   uint32_t tmem_base, EpiState& es, int rank, int quad, int lane,
                                                   const SwapWork& wk, int t, const WaitCtl& wc, const DEP& dep) {
  constexpr int SLOTB = swap_staging_slot_bytes<MODE>();
  uint8_t* sOut = smem + PIPE_STAGES * (W_STAGE_BYTES + tok_stage_bytes<MODE>());
  uint8_t* sScr = sOut + 4 * SW_SLOTS * SLOTB;   // act_grad: per epilogue warp 4 KB for the saved pre-activations
  SwStaging sg{sOut + quad * SW_SLOTS * SLOTB, es.round, sScr + quad * SW_SCRATCH_BYTES, SW_SLOTS, (uint32_t)SLOTB};
  bool ok = true;
  for (int part = 0; part < (wk.merged ? 2 : 1); ++part) {   // a merged item is two consecutive tiles here
    const SwapTile& st = part ? wk.b : wk.a;
    const int as = es.acc_it & 1;
    if (!mbar_wait(&bars->tmem_full[as], (es.acc_it >> 1) & 1, wc, SITE_TMEM_FULL, t, 200)) { ok = false; break; }
    uint64_t t0 = 0;
    if (DEP::kOn && quad == 0 && lane == 0 && dep.tracing()) t0 = globaltimer_ns();
    tc_fence_after_sync();
    epilogue_swap<MODE>(a, st, tmem_base + as * BN, rank, quad, lane, sg);
    tc_fence_before_sync();
    __syncwarp();
    if (lane == 0) mbar_arrive_leader(&bars->tmem_empty[as]);
    ++es.acc_it;
    if (DEP::kOn) {
      if (lane == 0) {
        tma_store_wait_all();
        fence_proxy_async();
        dep.signal(st.mb_first, st.mb_count);
        if (quad == 0 && dep.tracing()) dep.trace(TR_EPI, t, t0, t0, globaltimer_ns());
      }
      __syncwarp();
    }
  }
  es.round = sg.round;
  return ok;
}

// =====================================================================================================
// Weight gradients, strip by strip, the strip's A operand resident in shared memory
// =====================================================================================================
// dW[e] (M x N) = P_e^T . Q_e with K = the expert's rows: at a few hundred rows per expert a 256 x 256
// tile reads 320 KB of operands for 128 KB of output.  A pair therefore takes a whole strip (its 256
// rows of dW across all column tiles) and loads the strip's A operand (this CTA's 128 columns of P_e,
// all K rows) once: when the expert has at most A_RES_KB k-blocks it stays in the five 16 KB A slots for
// every column tile of the strip, and only the B operand streams through the stage ring.  Longer
// experts stream A through the same slots stage by stage.  An A slot is refilled only after the MMAs
// that read its previous content have completed (a_empty, one commit per content).
//
// With K of only four or five k-blocks a column tile lasts about as long as the latency of its B loads, so the
// B ring is deeper than one tile (WG_B_STAGES): the loads of tile i + 1 are in flight while tile i multiplies.
// The staging of the epilogue is what pays for it: one 4 KB box of 32 rows x 64 columns at a time, two per warp.
constexpr int A_RES_KB = PIPE_STAGES;        // k-blocks of A that can stay resident
constexpr int WG_OUT_SLOTS = 2;              // staging boxes per epilogue warp
constexpr size_t WGRAD_LAYOUT_BYTES =
    (size_t)PIPE_STAGES * A_STAGE_BYTES + (size_t)WG_B_STAGES * HALF_B_BYTES + 4 * WG_OUT_SLOTS * OUT_BOX_BYTES;

// Epilogue of one 128 x 256 accumulator slice of a weight gradient (or zeros for an expert without rows): warp
// `quad` stores its 32 rows, 64 columns per staging box.
__device__ __forceinline__ void epilogue_wgrad_tile(const GemmArgs& a, const Tile& tl, uint32_t tmem_acc, int quad, int lane,
                                                    uint8_t* slots, uint32_t& round) {
  const uint32_t trow = tmem_acc + (static_cast<uint32_t>(quad * 32) << 16);
  const int y0 = tl.m0 + quad * 32;
  if (y0 >= a.M) return;
#pragma unroll 1
  for (int c0 = 0; c0 < BN; c0 += 64) {
    if (tl.n0 + c0 >= a.N) break;
    float v[64];
    if (tl.nkb == 0) {
#pragma unroll
      for (int i = 0; i < 64; ++i) v[i] = 0.f;
    } else {
      // 64 columns per TMEM round trip (one wait per box)
#pragma unroll
      for (int q = 0; q < 4; ++q) tmem_ld16(trow + c0 + 16 * q, v + 16 * q);
      tmem_ld_wait();
    }
    if (lane == 0) tma_store_wait_read_n<WG_OUT_SLOTS - 1>();   // the box's previous store has read it
    __syncwarp();
    uint8_t* box = slots + (round % WG_OUT_SLOTS) * OUT_BOX_BYTES;
    ++round;
#pragma unroll
    for (int h = 0; h < 64; h += 8) stage8(box, lane, h >> 3, v + h);
    staging_release();
    if (lane == 0) {
      tma_store_3d(&a.tmOut0, tl.n0 + c0, y0, tl.e, box);
      tma_store_commit();
    }
  }
}

struct Strip {
  int e, mp, row0, nkb, rows;   // expert, 256-row block of dW, first padded row, k-blocks, rows of the expert
  bool resident;
  __device__ __forceinline__ int m0(int rank) const { return (2 * mp + rank) * BLOCK_M; }   // this CTA's 128 rows
};
__device__ __forceinline__ int wgrad_strips(const GemmArgs& a) { return a.Ep * ((a.n_tiles_m + 1) / 2); }
// Strip s of the operator: expert-major, so the pairs working at the same time share the expert's B operand
// in L2.
__device__ __forceinline__ Strip decode_strip(const GemmArgs& a, int s) {
  Strip st;
  const int tm2 = (a.n_tiles_m + 1) / 2;
  st.e = s / tm2;
  st.mp = s - st.e * tm2;
  st.row0 = a.mb_start[st.e] * BLOCK_M;
  st.rows = a.counts[st.e];
  st.nkb = (st.rows + BK - 1) / BK;
  st.resident = st.nkb <= A_RES_KB;
  return st;
}

// TMA producers (both CTAs) of strip sp.  b_warp = false: A (and the stage's byte count); true: B.
template <class DEP>
__device__ __forceinline__ bool wgrad_load_strip(const GemmArgs& a, uint8_t* smem, PipeBarriers* bars, LoaderState& ls,
                                                 bool b_warp, int rank, int lane, const Strip& st, int sp,
                                                 const WaitCtl& wc, const DEP& dep) {
  uint8_t* sA = smem;                                   // [PIPE_STAGES][16 KB] A slots
  uint8_t* sB = smem + PIPE_STAGES * A_STAGE_BYTES;     // [WG_B_STAGES][16 KB] B stages
  const int m0 = st.m0(rank);
  if (DEP::kOn) fence_proxy_async();   // as in swap_load_item
  for (int nb = 0; nb < a.n_tiles_n; ++nb) {
    const bool load_a = !st.resident || nb == 0;
    for (int kb = 0; kb < st.nkb; ++kb) {
      const int slot = st.resident ? kb : (int)ls.a_s;
      int go = 1;
      if (lane == 0) {
        go = mbar_wait(&bars->empty[ls.s], (ls.empty_par >> ls.s) & 1, wc, SITE_EMPTY, sp, 50) ? 1 : 0;
        if (go && !b_warp && load_a)
          go = mbar_wait(&bars->a_empty[slot], (ls.a_ph >> slot) & 1, wc, SITE_EMPTY, sp, 50) ? 1 : 0;
      }
      go = __shfl_sync(0xffffffffu, go, 0);
      if (!go) return false;
      const int k0 = kb * BK;
      if (!b_warp) {
        if (lane == 0 && rank == 0)
          mbar_expect_tx(&bars->full[ls.s], 2 * (HALF_B_BYTES + (load_a ? A_STAGE_BYTES : 0)));
        __syncwarp();
        if (load_a && lane < 2)
          tma_load_2d_pair(sA + slot * A_STAGE_BYTES + lane * MN_BOX_BYTES, &a.tmA, m0 + lane * 64, st.row0 + k0,
                           &bars->full[ls.s]);
      } else if (lane < 2) {
        tma_load_2d_pair(sB + ls.s * HALF_B_BYTES + lane * MN_BOX_BYTES, &a.tmB, nb * BN + (2 * rank + lane) * 64,
                         st.row0 + k0, &bars->full[ls.s]);
      }
      ls.empty_par ^= 1u << ls.s;
      if (load_a) ls.a_ph ^= 1u << slot;
      if (!st.resident && ++ls.a_s == PIPE_STAGES) ls.a_s = 0;
      if (++ls.s == WG_B_STAGES) ls.s = 0;
    }
  }
  return true;
}

template <class DEP>
__device__ __forceinline__ bool wgrad_issue_strip(const GemmArgs& a, uint8_t* smem, PipeBarriers* bars, uint32_t tmem_base,
                                                  IssuerState& is, bool issue, const Strip& st, int sp,
                                                  const WaitCtl& wc, const DEP& dep) {
  uint8_t* sA = smem;
  uint8_t* sB = smem + PIPE_STAGES * A_STAGE_BYTES;
  if (st.nkb == 0) return true;
  uint64_t t0 = 0;
  for (int nb = 0; nb < a.n_tiles_n; ++nb) {
    const int as = is.acc_it & 1;
    if (!mbar_wait(&bars->tmem_empty[as], ((is.acc_it >> 1) & 1) ^ 1, wc, SITE_TMEM_EMPTY, sp)) return false;
    tc_fence_after_sync();
    const uint32_t d_tmem = tmem_base + as * BN;
    const bool last_use = !st.resident || nb == a.n_tiles_n - 1;
    for (int kb = 0; kb < st.nkb; ++kb) {
      if (!mbar_wait(&bars->full[is.s], (is.full_par >> is.s) & 1, wc, SITE_FULL, sp)) return false;
      is.full_par ^= 1u << is.s;
      if (DEP::kOn && nb == 0 && kb == 0 && issue && dep.tracing()) t0 = globaltimer_ns();
      tc_fence_after_sync();
      const int slot = st.resident ? kb : (int)is.a_s;
      if (issue) {
        mma_kblock_pair<GEMM_WGRAD>(d_tmem, smem_u32(sA + slot * A_STAGE_BYTES), smem_u32(sB + is.s * HALF_B_BYTES),
                                    kb == 0, k16_steps_of(st.rows, kb));
        tc_commit_pair(&bars->empty[is.s]);
        if (last_use) tc_commit_pair(&bars->a_empty[slot]);
      }
      if (!st.resident && ++is.a_s == PIPE_STAGES) is.a_s = 0;
      if (++is.s == WG_B_STAGES) is.s = 0;
    }
    if (issue) tc_commit_pair(&bars->tmem_full[as]);
    ++is.acc_it;
  }
  if (DEP::kOn && issue && dep.tracing()) dep.trace(TR_MMA, sp, t0, t0, globaltimer_ns());
  return true;
}

template <class DEP>
__device__ __forceinline__ bool wgrad_epilogue_strip(const GemmArgs& a, uint8_t* smem, PipeBarriers* bars,
                                                     uint32_t tmem_base, EpiState& es, int rank, int quad, int lane,
                                                     const Strip& st, int sp, const WaitCtl& wc, const DEP& dep) {
  uint8_t* slots = smem + PIPE_STAGES * A_STAGE_BYTES + WG_B_STAGES * HALF_B_BYTES + quad * WG_OUT_SLOTS * OUT_BOX_BYTES;
  Tile tl;
  tl.e = st.e; tl.row0 = st.row0; tl.m0 = st.m0(rank); tl.nkb = st.nkb;
  const bool idle = tl.m0 >= a.M;   // the strip's second half lies outside dW: nothing to store
  bool ok = true;
  uint64_t t0 = 0;
  if (DEP::kOn && quad == 0 && lane == 0 && dep.tracing()) t0 = globaltimer_ns();
  for (int nb = 0; nb < a.n_tiles_n; ++nb) {
    tl.nb = nb; tl.n0 = nb * BN;
    if (st.nkb == 0) {
      if (!idle) epilogue_wgrad_tile(a, tl, 0, quad, lane, slots, es.round);  // an expert without rows: zeros
      continue;
    }
    const int as = es.acc_it & 1;
    if (!mbar_wait(&bars->tmem_full[as], (es.acc_it >> 1) & 1, wc, SITE_TMEM_FULL, sp, 200)) { ok = false; break; }
    tc_fence_after_sync();
    if (!idle) epilogue_wgrad_tile(a, tl, tmem_base + as * BN, quad, lane, slots, es.round);
    tc_fence_before_sync();
    __syncwarp();
    if (lane == 0) mbar_arrive_leader(&bars->tmem_empty[as]);
    ++es.acc_it;
  }
  if (DEP::kOn && quad == 0 && lane == 0 && dep.tracing()) dep.trace(TR_EPI, sp, t0, t0, globaltimer_ns());
  return ok;
}

}  // namespace moe
