// Scheduling microbenchmarks on a SwiGLU + Add operator pair (Section 6): the same two element-wise
// operators, split into row tiles, run three ways --
//   serial    one kernel per operator: SwiGLU finishes all rows before Add begins (the baseline of Section 6.1);
//   static    one persistent launch, statically ordered task lists per worker, event counters with static
//             thresholds: worker b runs SwiGLU of tile i*G+b and then Add of the tile its neighbour produced
//             one round earlier, so every intermediate tile is consumed by another SM shortly after it was
//             written, through L2 (Section 6.1 "interleaved", Section 6.2 "static");
//   dynamic   the same tasks and events, but dispatched at run time: producer tasks from a ticket, consumer
//             tasks from a FIFO ready queue in global memory that a finished producer appends to and that a
//             free worker pops first (Section 6.2 "dynamic").
// s = silu(gate) * up is stored in bf16 between the operators in every mode.  Each worker also accounts the
// time between the end of one task's work and the start of the next one's (ticket, decode, queue and event
// waits): the per-task dispatch cost the paper compares.
#include "../../include/moe_b200.h"
#include "moe_internal.h"
#include "study_ops.cuh"

namespace moe {

constexpr int STUDY_WORKERS_PER_SM = 4;
// workspace (ints): status word, queue head / tail, dispatch accounting, one event counter per tile, the queue
constexpr int SW_STATUS = 0, SW_HEAD = 4, SW_TAIL = 5, SW_STICKET = 6, SW_STATS = 8 /* 2 x u64 */, SW_EVENTS = 16;

// ---------------------------------------------------------------- serial: one kernel per operator
__global__ void __launch_bounds__(STUDY_THREADS, 4) study_swiglu_kernel(const uint16_t* x, uint16_t* s, int M, int C, int tile_rows) {
  const int ntiles = (M + tile_rows - 1) / tile_rows;
  for (int t = blockIdx.x; t < ntiles; t += gridDim.x) swiglu_tile<SERIAL_UNROLL>(x, s, C, t * tile_rows, min(M, (t + 1) * tile_rows));
}
__global__ void __launch_bounds__(STUDY_THREADS, 4) study_add_kernel(const uint16_t* s, const uint16_t* r, uint16_t* z, int M, int C,
                                                                   int tile_rows) {
  const int ntiles = (M + tile_rows - 1) / tile_rows;
  for (int t = blockIdx.x; t < ntiles; t += gridDim.x) add_tile<SERIAL_UNROLL>(s, r, z, C, t * tile_rows, min(M, (t + 1) * tile_rows));
}

// ---------------------------------------------------------------- persistent launches
struct StudyArgs {
  const uint16_t* x;
  const uint16_t* r;
  uint16_t* s;
  uint16_t* z;
  int M, C, tile_rows, ntiles;
  int* ws;
  uint64_t budget_ns;
};

// Worker-side accounting: dispatch time = everything between the end of a task's work and the start of the next.
struct Dispatch {
  uint64_t t_mark, sum;
  unsigned n;
};
__device__ __forceinline__ void dispatch_done(Dispatch& d) {   // thread 0, right before a task's work starts
  const uint64_t now = globaltimer_ns();
  d.sum += now - d.t_mark;
  ++d.n;
}
__device__ __forceinline__ void work_done(Dispatch& d) { d.t_mark = globaltimer_ns(); }   // thread 0, after the work

__device__ __forceinline__ void study_flush(const StudyArgs& a, const Dispatch& d) {
  unsigned long long* st = reinterpret_cast<unsigned long long*>(a.ws + SW_STATS);
  atomicAdd(&st[0], (unsigned long long)d.sum);
  atomicAdd(&st[1], (unsigned long long)d.n);
}

// The producer's trigger event: after the block's stores of the tile.
__device__ __forceinline__ void tile_signal(const StudyArgs& a, int tile) {
  __syncthreads();
  if (threadIdx.x == 0) counter_signal(a.ws + SW_EVENTS + tile, 1);
}
// The consumer's dependent event (threshold 1).  Returns false after a timeout / abort (all threads agree).
__device__ __forceinline__ bool tile_wait(const StudyArgs& a, int tile, const WaitCtl& wc) {
  __shared__ int ok_s;
  if (threadIdx.x == 0) ok_s = counter_wait(a.ws + SW_EVENTS + tile, 1, wc, tile, 256) ? 1 : 0;
  __syncthreads();
  const int ok = ok_s;
  __syncthreads();
  return ok != 0;
}

// static: worker b of G, round i: SwiGLU(tile i*G + b), then Add(tile (i-1)*G + (b+1) % G); one closing round of Adds.
__global__ void __launch_bounds__(STUDY_THREADS, STUDY_WORKERS_PER_SM) study_static_kernel(const StudyArgs a) {
  const WaitCtl wc{reinterpret_cast<DevStatus*>(a.ws + SW_STATUS), a.budget_ns};
  const int G = gridDim.x, b = blockIdx.x;
  const int rounds = (a.ntiles + G - 1) / G;
  Dispatch d{0, 0, 0};
  if (threadIdx.x == 0) d.t_mark = globaltimer_ns();
  for (int i = 0; i <= rounds; ++i) {
    const int ts = i * G + b;
    if (i < rounds && ts < a.ntiles) {
      if (threadIdx.x == 0) dispatch_done(d);
      swiglu_tile<WORKER_UNROLL>(a.x, a.s, a.C, ts * a.tile_rows, min(a.M, (ts + 1) * a.tile_rows));
      tile_signal(a, ts);
      if (threadIdx.x == 0) work_done(d);
    }
    const int ta = (i - 1) * G + (b + 1) % G;
    if (i >= 1 && ta < a.ntiles) {
      if (!tile_wait(a, ta, wc)) break;
      if (threadIdx.x == 0) dispatch_done(d);
      add_tile<WORKER_UNROLL>(a.s, a.r, a.z, a.C, ta * a.tile_rows, min(a.M, (ta + 1) * a.tile_rows));
      __syncthreads();
      if (threadIdx.x == 0) work_done(d);
    }
  }
  if (threadIdx.x == 0) study_flush(a, d);
}

// dynamic: nothing is ordered ahead of time.  Producer tasks (SwiGLU tiles) are handed out by a ticket; a finished
// producer appends its consumer task (Add of the same tile) to a FIFO ready queue in global memory.  A free worker
// that sees a published entry claims the next slot of the queue, else takes the next producer ticket, and once the
// producers are handed out it claims queue slots in order and waits for each to be published.
__global__ void __launch_bounds__(STUDY_THREADS, STUDY_WORKERS_PER_SM) study_dynamic_kernel(const StudyArgs a) {
  const WaitCtl wc{reinterpret_cast<DevStatus*>(a.ws + SW_STATUS), a.budget_ns};
  int* queue = a.ws + SW_EVENTS + a.ntiles;   // ready queue: entry = tile + 1; 0 = reserved but not yet published
  int* head = a.ws + SW_HEAD;
  int* tail = a.ws + SW_TAIL;
  __shared__ int task_s;
  Dispatch d{0, 0, 0};
  bool producers_left = true;   // thread 0's view
  if (threadIdx.x == 0) d.t_mark = globaltimer_ns();
  while (true) {
    if (threadIdx.x == 0) {
      int task = -1, slot = -1;
      int h = *reinterpret_cast<volatile int*>(head), t;
      asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(t) : "l"(tail) : "memory");
      // A consumer task looks ready: claim the next slot.  Several workers may claim on the same observation; the
      // ones past the tail wait for the next producers to publish (a retry loop of compare-and-swap instead lets
      // one contender through per round trip to L2 and is an order of magnitude slower with hundreds of workers).
      if (h < t) {
        const int c = atomicAdd(head, 1);
        if (c < a.ntiles) slot = c;   // else: every consumer is claimed; producer tickets may still be left
      }
      if (slot < 0) {
        const int p = producers_left ? atomicAdd(a.ws + SW_STICKET, 1) : a.ntiles;
        if (p < a.ntiles) task = p;
        else {
          producers_left = false;
          const int c = atomicAdd(head, 1);   // every producer is handed out: the remaining work is in the queue
          if (c < a.ntiles) slot = c;
        }
      }
      if (slot >= 0)
        task = counter_wait(queue + slot, 1, wc, slot, 256) ? a.ntiles + *reinterpret_cast<volatile int*>(queue + slot) - 1 : -2;
      task_s = task;
    }
    __syncthreads();
    const int task = task_s;
    __syncthreads();
    if (task < 0) break;
    if (task < a.ntiles) {
      if (threadIdx.x == 0) dispatch_done(d);
      swiglu_tile<WORKER_UNROLL>(a.x, a.s, a.C, task * a.tile_rows, min(a.M, (task + 1) * a.tile_rows));
      tile_signal(a, task);
      if (threadIdx.x == 0) {
        work_done(d);
        const int slot = atomicAdd(tail, 1);   // reserve, then publish the consumer task
        asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(queue + slot), "r"(task + 1) : "memory");
      }
    } else {
      const int tile = task - a.ntiles;
      if (!tile_wait(a, tile, wc)) break;   // the same dependent event as the static schedule (already met here)
      if (threadIdx.x == 0) dispatch_done(d);
      add_tile<WORKER_UNROLL>(a.s, a.r, a.z, a.C, tile * a.tile_rows, min(a.M, (tile + 1) * a.tile_rows));
      __syncthreads();
      if (threadIdx.x == 0) work_done(d);
    }
  }
  if (threadIdx.x == 0) study_flush(a, d);
}

std::atomic<bool>& study_plain_launch() {
  static std::atomic<bool> flag{false};
  return flag;
}

}  // namespace moe

using namespace moe;

extern "C" {

size_t moe_sched_study_workspace_bytes(int32_t M, int32_t tile_rows) {
  if (M < 0 || tile_rows < 1) return 0;
  const size_t ntiles = ((size_t)M + tile_rows - 1) / tile_rows;
  return sizeof(int) * (SW_EVENTS + 3 * ntiles + 16);
}

int moe_sched_study(int32_t mode, const uint16_t* x, const uint16_t* r, uint16_t* s, uint16_t* z, int32_t M, int32_t C,
                    int32_t tile_rows, void* workspace, size_t workspace_bytes, void* stream) {
  if (!workspace || M < 0 || C < 8 || C % 8 != 0 || tile_rows < 1 || mode < 0 || mode > 2)
    return MOE_ERR_INVALID_ARG;
  if (workspace_bytes < moe_sched_study_workspace_bytes(M, tile_rows) || (reinterpret_cast<uintptr_t>(workspace) & 15))
    return MOE_ERR_WORKSPACE;
  if (M > 0 && (!x || !r || !s || !z ||
                ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(r) | reinterpret_cast<uintptr_t>(s) |
                  reinterpret_cast<uintptr_t>(z)) & 15) != 0))
    return MOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int dev = 0, sms = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOE_ERR_NO_DEVICE;
  cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (major != 10) return MOE_ERR_NO_DEVICE;
  StudyArgs a;
  a.x = x; a.r = r; a.s = s; a.z = z; a.M = M; a.C = C; a.tile_rows = tile_rows;
  a.ntiles = (M + tile_rows - 1) / tile_rows;
  a.ws = static_cast<int*>(workspace);
  a.budget_ns = 2000ull * 1000 * 1000;
  if (cudaMemsetAsync(workspace, 0, moe_sched_study_workspace_bytes(M, tile_rows), st) != cudaSuccess) return MOE_ERR_CUDA;
  if (M == 0) return MOE_OK;
  const int workers = STUDY_WORKERS_PER_SM * sms;   // all resident (the launch bound caps the registers for it)
  if (mode == 0) {
    const int grid = a.ntiles < 8 * sms ? a.ntiles : 8 * sms;
    study_swiglu_kernel<<<grid, STUDY_THREADS, 0, st>>>(x, s, M, C, tile_rows);
    study_add_kernel<<<grid, STUDY_THREADS, 0, st>>>(s, r, z, M, C, tile_rows);
    return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
  }
  void* params[] = {&a};
  // cooperative: the launch fails rather than run with workers that are not all resident (consumers wait for producers)
  const void* fn = mode == 1 ? reinterpret_cast<const void*>(study_static_kernel) : reinterpret_cast<const void*>(study_dynamic_kernel);
  const int grid = a.ntiles < workers ? a.ntiles : workers;
  cudaError_t e = study_plain_launch().load() ? cudaLaunchKernel(fn, dim3(grid), dim3(STUDY_THREADS), params, 0, st)
                                              : cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(STUDY_THREADS), params, 0, st);
  return e == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

int moe_sched_study_stats(const void* workspace, int32_t* status2, uint64_t* dispatch_ns, uint64_t* tasks, void* stream) {
  if (!workspace) return MOE_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return MOE_ERR_CUDA;
  int head[16];
  if (cudaMemcpy(head, workspace, sizeof head, cudaMemcpyDeviceToHost) != cudaSuccess) return MOE_ERR_CUDA;
  if (status2) { status2[0] = head[SW_STATUS]; status2[1] = head[SW_STATUS + 1]; }
  const unsigned long long* st = reinterpret_cast<const unsigned long long*>(head + SW_STATS);
  if (dispatch_ns) *dispatch_ns = st[0];
  if (tasks) *tasks = st[1];
  return MOE_OK;
}

}  // extern "C"
