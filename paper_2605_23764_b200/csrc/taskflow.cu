// Generic taskflow front end and its device runtime (Section 4.2: Operator Dependency Graph, SplitSpec, split
// propagation -- Algorithm 1 --, FillConfig and the Task Descriptor of Table 1; Section 4.3: statically ordered
// queues, events with static thresholds; Section 4.4: workers that fetch the next descriptor, wait, dispatch on
// task_type, trigger).  The host part compiles a graph of element-wise operators into descriptors; the device part
// is a persistent kernel that interprets descriptors and knows nothing about the graph they came from.
#include <algorithm>
#include <queue>
#include <vector>

#include "../../include/moe_b200.h"
#include "moe_internal.h"
#include "study_ops.cuh"

namespace moe {

// ---------------------------------------------------------------- host: graph -> descriptors
namespace {

struct UnionFind {
  std::vector<int> p;
  explicit UnionFind(int n) : p(n) { for (int i = 0; i < n; ++i) p[i] = i; }
  int find(int a) { while (p[a] != a) a = p[a] = p[p[a]]; return a; }
  void unite(int a, int b) { p[find(a)] = find(b); }
};

bool shapes_ok(const moe_tf_tensor* ts, int nt, const moe_tf_operator& op) {
  auto id_ok = [&](int t) { return t >= 0 && t < nt; };
  if (op.n_inputs < 1 || op.n_inputs > 4 || op.n_outputs < 1 || op.n_outputs > 2 || op.task_rows < 1) return false;
  for (int i = 0; i < op.n_inputs; ++i) if (!id_ok(op.inputs[i])) return false;
  for (int j = 0; j < op.n_outputs; ++j) if (!id_ok(op.outputs[j])) return false;
  if (op.n_split_inputs < -1 || op.n_split_inputs > 4) return false;
  for (int i = 0; i < op.n_split_inputs; ++i)
    if (op.split_input_idx[i] < 0 || op.split_input_idx[i] >= op.n_inputs) return false;
  for (int j = 0; j < op.n_outputs; ++j)
    if (op.split_output_dim[j] != -1 && op.split_output_dim[j] != 0) return false;   // the handlers split rows only
  const moe_tf_tensor& o = ts[op.outputs[0]];
  if (o.rows < 0 || o.cols < 8 || o.cols % 8) return false;
  if (op.op == MOE_TF_SWIGLU) {
    const moe_tf_tensor& x = ts[op.inputs[0]];
    return op.n_inputs == 1 && op.n_outputs == 1 && x.rows == o.rows && x.cols == 2 * o.cols;
  }
  if (op.op == MOE_TF_ADD) {
    if (op.n_inputs != 2 || op.n_outputs != 1) return false;
    for (int i = 0; i < 2; ++i)
      if (ts[op.inputs[i]].rows != o.rows || ts[op.inputs[i]].cols != o.cols) return false;
    return true;
  }
  return false;
}

}  // namespace

int taskflow_compile(const moe_tf_tensor* ts, int nt, const moe_tf_operator* ops, int nops, int lag_rows,
                     std::vector<moe_tf_td>& out, int* n_events, int* op_task_num, int* t_split_dim, int* t_split_num) {
  if (nt < 1 || nops < 1 || lag_rows < 0) return MOE_ERR_INVALID_ARG;
  std::vector<int> producer(nt, -1);
  for (int o = 0; o < nops; ++o) {
    if (!shapes_ok(ts, nt, ops[o])) return MOE_ERR_INVALID_ARG;
    for (int j = 0; j < ops[o].n_outputs; ++j) {
      if (producer[ops[o].outputs[j]] != -1) return MOE_ERR_INVALID_ARG;   // two writers of one tensor
      producer[ops[o].outputs[j]] = o;
    }
  }
  // topological order of the operators (Kahn), and the depth of each (longest chain of producers behind it)
  std::vector<int> indeg(nops, 0), depth(nops, 0), topo;
  std::vector<std::vector<int>> users(nops);
  for (int o = 0; o < nops; ++o)
    for (int i = 0; i < ops[o].n_inputs; ++i) {
      const int p = producer[ops[o].inputs[i]];
      if (p == o) return MOE_ERR_INVALID_ARG;
      if (p >= 0) { users[p].push_back(o); ++indeg[o]; }
    }
  for (int o = 0; o < nops; ++o) if (indeg[o] == 0) topo.push_back(o);
  for (size_t h = 0; h < topo.size(); ++h)
    for (int u : users[topo[h]]) {
      depth[u] = std::max(depth[u], depth[topo[h]] + 1);
      if (--indeg[u] == 0) topo.push_back(u);
    }
  if ((int)topo.size() != nops) return MOE_ERR_INVALID_ARG;   // a cycle

  // ---- split propagation (Algorithm 1): labels live on tensors, written by producers, checked by consumers
  std::vector<int> split_dim(nt, -1), split_num(nt, 1), task_num(nops, 1);
  for (int o : topo) {
    const moe_tf_operator& op = ops[o];
    const int rows = ts[op.outputs[0]].rows;
    const int by_fn = std::max(1, (rows + op.task_rows - 1) / op.task_rows);   // task_num_fn of this shape
    int n;
    if (op.n_split_inputs < 0) {
      n = by_fn;                                        // split_inputs = None: a partition origin
    } else {
      bool inherits = true;
      for (int i = 0; i < op.n_split_inputs; ++i)
        if (split_dim[op.inputs[op.split_input_idx[i]]] != op.split_input_dim[i]) inherits = false;
      n = inherits ? by_fn : 1;                         // otherwise: one unsplit task
    }
    task_num[o] = n;
    for (int j = 0; j < op.n_outputs; ++j) {
      const int d = op.split_output_dim[j];
      split_dim[op.outputs[j]] = (n > 1 && d >= 0) ? d : -1;
      split_num[op.outputs[j]] = n;
    }
  }
  // rows one task of an operator covers
  auto rows_per_task = [&](int o) { return task_num[o] > 1 ? ops[o].task_rows : std::max(1, ts[ops[o].outputs[0]].rows); };

  // ---- events.  A descriptor has ONE dependent and ONE trigger event (Table 1), so:
  //  - the outputs of one operator share a family of counters (one counter per row block);
  //  - an operator with several produced inputs waits on the input whose producer has the producers of all the
  //    others among its ancestors: every operator here is row-local, so when a row block of that input is
  //    complete, the same rows of its ancestors' outputs were complete before it;
  //  - if no input dominates the others like that, the inputs share one family of counters that all their
  //    producers raise (many producers, one event, threshold = their number: Section 4.3).
  std::vector<std::vector<char>> ancestor(nops, std::vector<char>(nops, 0));   // ancestor[o][a]: a is upstream of o
  for (int o : topo)
    for (int i = 0; i < ops[o].n_inputs; ++i) {
      const int p = producer[ops[o].inputs[i]];
      if (p < 0) continue;
      ancestor[o][p] = 1;
      for (int a = 0; a < nops; ++a) if (ancestor[p][a]) ancestor[o][a] = 1;
    }
  UnionFind uf(nt);
  std::vector<char> consumed(nt, 0);
  std::vector<int> dep_tensor(nops, -1);
  for (int o = 0; o < nops; ++o) {
    std::vector<int> produced;
    for (int i = 0; i < ops[o].n_inputs; ++i)
      if (producer[ops[o].inputs[i]] >= 0) produced.push_back(ops[o].inputs[i]);
    for (int j = 1; j < ops[o].n_outputs; ++j) uf.unite(ops[o].outputs[0], ops[o].outputs[j]);
    if (produced.empty()) continue;
    int dominant = -1;
    for (int t : produced) {
      bool all = true;
      for (int u : produced)
        if (producer[u] != producer[t] && !ancestor[producer[t]][producer[u]]) all = false;
      if (all) { dominant = t; break; }
    }
    if (dominant >= 0) {
      dep_tensor[o] = dominant;
      consumed[dominant] = 1;
    } else {
      for (int t : produced) { consumed[t] = 1; uf.unite(produced[0], t); }
      dep_tensor[o] = produced[0];
    }
  }
  std::vector<int> grp_rows(nt, -1), grp_gran(nt, 0), grp_base(nt, -1), grp_used(nt, 0);
  auto touch = [&](int t, int o) -> bool {   // operator o reads or writes produced tensor t
    const int g = uf.find(t);
    if (grp_rows[g] < 0) grp_rows[g] = ts[t].rows;
    if (grp_rows[g] != ts[t].rows) return false;
    grp_gran[g] = std::max(grp_gran[g], rows_per_task(o));
    return true;
  };
  for (int o = 0; o < nops; ++o) {
    if (dep_tensor[o] >= 0 && !touch(dep_tensor[o], o)) return MOE_ERR_INVALID_ARG;
    for (int j = 0; j < ops[o].n_outputs; ++j)
      if (!touch(ops[o].outputs[j], o)) return MOE_ERR_INVALID_ARG;
  }
  for (int t = 0; t < nt; ++t)
    if (consumed[t]) grp_used[uf.find(t)] = 1;
  int nev = 0;
  for (int t = 0; t < nt; ++t) {
    const int g = uf.find(t);
    if (g != t || !grp_used[g]) continue;
    grp_base[g] = nev;
    nev += std::max(1, (grp_rows[g] + grp_gran[g] - 1) / std::max(1, grp_gran[g]));
  }
  auto nests = [&](int g, int o) {   // a task of o lies inside one block of g
    const int r = rows_per_task(o);
    return grp_gran[g] % r == 0 || grp_gran[g] >= grp_rows[g];
  };
  std::vector<int> dep_grp(nops, -1), trig_grp(nops, -1);
  for (int o = 0; o < nops; ++o) {
    if (dep_tensor[o] >= 0) dep_grp[o] = uf.find(dep_tensor[o]);
    const int g = uf.find(ops[o].outputs[0]);
    if (grp_used[g]) trig_grp[o] = g;
    if (dep_grp[o] >= 0 && dep_grp[o] == trig_grp[o]) return MOE_ERR_INVALID_ARG;   // would wait for its own trigger
    if (dep_grp[o] >= 0 && !nests(dep_grp[o], o)) return MOE_ERR_INVALID_ARG;
    if (trig_grp[o] >= 0 && !nests(trig_grp[o], o)) return MOE_ERR_INVALID_ARG;
  }

  // ---- FillConfig: one descriptor per task
  std::vector<moe_tf_td> tds;
  std::vector<double> key;
  std::vector<int> threshold(std::max(nev, 1), 0);
  for (int oi = 0; oi < nops; ++oi) {
    const int o = topo[oi];
    const moe_tf_operator& op = ops[o];
    const int rows = ts[op.outputs[0]].rows, per = rows_per_task(o);
    for (int i = 0; i < task_num[o]; ++i) {
      moe_tf_td td;
      memset(&td, 0, sizeof td);
      const int r0 = i * per, nr = std::max(0, std::min(per, rows - r0));
      td.task_type = (uint32_t)op.op;
      td.queue_type = MOE_TF_QUEUE_VECTOR;             // both handlers of this build are element-wise
      td.task_index = (uint32_t)i;
      td.task_split_num = (uint32_t)task_num[o];
      td.task_split_value = (uint32_t)per;
      td.tiling_data_position = (uint32_t)o;
      td.n_inputs = (uint32_t)op.n_inputs;
      td.n_outputs = (uint32_t)op.n_outputs;
      for (int k = 0; k < op.n_inputs; ++k)
        td.inputs[k] = moe_tf_tdesc{(uint32_t)op.inputs[k], (uint32_t)r0, (uint32_t)nr, (uint32_t)ts[op.inputs[k]].cols};
      for (int k = 0; k < op.n_outputs; ++k)
        td.outputs[k] = moe_tf_tdesc{(uint32_t)op.outputs[k], (uint32_t)r0, (uint32_t)nr, (uint32_t)ts[op.outputs[k]].cols};
      td.dependent_event = dep_grp[o] >= 0 ? (uint32_t)(grp_base[dep_grp[o]] + r0 / grp_gran[dep_grp[o]]) : MOE_TF_NO_EVENT;
      td.trigger_event = trig_grp[o] >= 0 ? (uint32_t)(grp_base[trig_grp[o]] + r0 / grp_gran[trig_grp[o]]) : MOE_TF_NO_EVENT;
      if (td.trigger_event != MOE_TF_NO_EVENT) ++threshold[td.trigger_event];
      tds.push_back(td);
      key.push_back((double)r0 + (double)depth[o] * (double)lag_rows + 1e-6 * oi);
    }
  }
  for (moe_tf_td& td : tds)
    if (td.dependent_event != MOE_TF_NO_EVENT) td.dependent_threshold = (uint32_t)threshold[td.dependent_event];

  // ---- static order of the queue: by key, but never a task before the producers of its event (Section 4.3:
  // the order among independent tasks is free; Section 4.5 uses that freedom for locality)
  const int n = (int)tds.size();
  std::vector<std::vector<int>> waiters(std::max(nev, 1));
  std::vector<int> raised(std::max(nev, 1), 0);
  using Item = std::pair<double, int>;
  std::priority_queue<Item, std::vector<Item>, std::greater<Item>> ready;
  for (int i = 0; i < n; ++i) {
    if (tds[i].dependent_event == MOE_TF_NO_EVENT || tds[i].dependent_threshold == 0) ready.push({key[i], i});
    else waiters[tds[i].dependent_event].push_back(i);
  }
  out.clear();
  while (!ready.empty()) {
    const int i = ready.top().second;
    ready.pop();
    out.push_back(tds[i]);
    const uint32_t ev = tds[i].trigger_event;
    if (ev != MOE_TF_NO_EVENT && ++raised[ev] == threshold[ev])
      for (int w : waiters[ev]) ready.push({key[w], w});
  }
  if ((int)out.size() != n) return MOE_ERR_INVALID_ARG;
  *n_events = nev;
  for (int o = 0; o < nops; ++o) if (op_task_num) op_task_num[o] = task_num[o];
  for (int t = 0; t < nt; ++t) {
    if (t_split_dim) t_split_dim[t] = split_dim[t];
    if (t_split_num) t_split_num[t] = split_num[t];
  }
  return MOE_OK;
}

// ---------------------------------------------------------------- device: the descriptor runtime
constexpr int TF_STATUS = 0, TF_TICKET = 4, TF_MAGIC = 8, TF_EVENTS = 16;   // workspace ints
constexpr int TF_WORKERS_PER_SM = 4;

struct TfArgs {
  const moe_tf_td* tds;
  int n_tds;
  void* const* slots;
  int* ws;
  int magic;   // what an upload of this plan left at ws[TF_MAGIC]
  uint64_t budget_ns;
};

__device__ __forceinline__ uint16_t* tf_rows(const TfArgs& a, const moe_tf_tdesc& d) {
  return static_cast<uint16_t*>(a.slots[d.slot]);
}

// Workers take the next descriptor of the queue, wait for its dependent event, run its handler, raise its trigger.
__global__ void __launch_bounds__(STUDY_THREADS, TF_WORKERS_PER_SM) taskflow_kernel(const TfArgs a) {
  const WaitCtl wc{reinterpret_cast<DevStatus*>(a.ws + TF_STATUS), a.budget_ns};
  int* events = a.ws + TF_EVENTS;
  __shared__ int next_s, ok_s;
  // a run without upload on a workspace that does not hold this plan would interpret whatever is there: refuse
  if (*reinterpret_cast<volatile int*>(a.ws + TF_MAGIC) != a.magic) {
    if (threadIdx.x == 0) report(wc.status, MOE_ERR_BAD_EXPERT_ID, a.n_tds);
    return;
  }
  while (true) {
    if (threadIdx.x == 0) next_s = atomicAdd(a.ws + TF_TICKET, 1);
    __syncthreads();
    const int t = next_s;
    if (t >= a.n_tds) break;
    const moe_tf_td& td = a.tds[t];
    if (threadIdx.x == 0)
      ok_s = (td.dependent_event == MOE_TF_NO_EVENT ||
              counter_wait(events + td.dependent_event, (int)td.dependent_threshold, wc, t, 256)) ? 1 : 0;
    __syncthreads();
    if (!ok_s) break;
    const int r0 = (int)td.outputs[0].row_offset, r1 = r0 + (int)td.outputs[0].rows, C = (int)td.outputs[0].cols;
    // inputs may have been written earlier in this launch by another SM: read them at L2
    if (td.task_type == MOE_TF_SWIGLU)
      swiglu_tile<WORKER_UNROLL, true>(tf_rows(a, td.inputs[0]), tf_rows(a, td.outputs[0]), C, r0, r1);
    else if (td.task_type == MOE_TF_ADD)
      add_tile<WORKER_UNROLL, true>(tf_rows(a, td.inputs[0]), tf_rows(a, td.inputs[1]), tf_rows(a, td.outputs[0]), C, r0, r1);
    __syncthreads();   // the block's stores, then one release-increment; also protects next_s / ok_s
    if (threadIdx.x == 0 && td.trigger_event != MOE_TF_NO_EVENT) counter_signal(events + td.trigger_event, 1);
  }
}

}  // namespace moe

using namespace moe;

extern "C" {

int moe_taskflow_compile(const moe_tf_tensor* tensors, int32_t n_tensors, const moe_tf_operator* ops, int32_t n_ops,
                         int32_t lag_rows, moe_tf_td* tds, int32_t td_cap, int32_t* n_tds, int32_t* n_events,
                         int32_t* op_task_num, int32_t* tensor_split_dim, int32_t* tensor_split_num) {
  if (!tensors || !ops || !n_tds || !n_events || td_cap < 0) return MOE_ERR_INVALID_ARG;
  std::vector<moe_tf_td> out;
  int nev = 0;
  const int rc = taskflow_compile(tensors, n_tensors, ops, n_ops, lag_rows, out, &nev, op_task_num, tensor_split_dim,
                                  tensor_split_num);
  if (rc) return rc;
  *n_tds = (int32_t)out.size();
  *n_events = nev;
  if ((int)out.size() > td_cap || (!tds && !out.empty())) return MOE_ERR_WORKSPACE;
  for (size_t i = 0; i < out.size(); ++i) tds[i] = out[i];
  return MOE_OK;
}

static size_t tf_slots_offset(int n_events) { return (sizeof(int) * (size_t)(TF_EVENTS + n_events) + 15) & ~(size_t)15; }
static size_t tf_tds_offset(int n_events, int n_tensors) {
  return (tf_slots_offset(n_events) + sizeof(void*) * (size_t)n_tensors + 15) & ~(size_t)15;
}

size_t moe_taskflow_workspace_bytes(int32_t n_tds, int32_t n_events, int32_t n_tensors) {
  if (n_tds < 0 || n_events < 0 || n_tensors < 0) return 0;
  return tf_tds_offset(n_events, n_tensors) + sizeof(moe_tf_td) * (size_t)n_tds + 16;
}

int moe_taskflow_run(const moe_tf_td* tds, int32_t n_tds, int32_t n_events, void* const* slots, int32_t n_tensors,
                     void* workspace, size_t workspace_bytes, int32_t upload, void* stream) {
  if (!tds || !slots || !workspace || n_tds < 0 || n_events < 0 || n_tensors < 1) return MOE_ERR_INVALID_ARG;
  if (workspace_bytes < moe_taskflow_workspace_bytes(n_tds, n_events, n_tensors) || (reinterpret_cast<uintptr_t>(workspace) & 15))
    return MOE_ERR_WORKSPACE;
  for (int i = 0; i < n_tds; ++i) {   // a descriptor that points outside the slot table or at a misaligned tensor is refused here
    const moe_tf_td& td = tds[i];
    if (td.n_inputs > 4 || td.n_outputs < 1 || td.n_outputs > 2) return MOE_ERR_INVALID_ARG;
    if ((td.dependent_event != MOE_TF_NO_EVENT && td.dependent_event >= (uint32_t)n_events) ||
        (td.trigger_event != MOE_TF_NO_EVENT && td.trigger_event >= (uint32_t)n_events))
      return MOE_ERR_INVALID_ARG;
    for (uint32_t k = 0; k < td.n_inputs; ++k)
      if (td.inputs[k].slot >= (uint32_t)n_tensors || !slots[td.inputs[k].slot] ||
          (reinterpret_cast<uintptr_t>(slots[td.inputs[k].slot]) & 15) || td.inputs[k].cols % 8)
        return MOE_ERR_INVALID_ARG;
    for (uint32_t k = 0; k < td.n_outputs; ++k)
      if (td.outputs[k].slot >= (uint32_t)n_tensors || !slots[td.outputs[k].slot] ||
          (reinterpret_cast<uintptr_t>(slots[td.outputs[k].slot]) & 15) || td.outputs[k].cols % 8)
        return MOE_ERR_INVALID_ARG;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int dev = 0, sms = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOE_ERR_NO_DEVICE;
  cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (major != 10) return MOE_ERR_NO_DEVICE;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  // counters, ticket and status start at zero in every run; the plan mark between them stays
  if (cudaMemsetAsync(ws, 0, sizeof(int) * TF_MAGIC, st) != cudaSuccess) return MOE_ERR_CUDA;
  if (cudaMemsetAsync(ws + sizeof(int) * TF_EVENTS, 0, tf_slots_offset(n_events) - sizeof(int) * TF_EVENTS, st) != cudaSuccess)
    return MOE_ERR_CUDA;
  if (n_tds == 0) return MOE_OK;
  // the mark of this plan: its sizes, the slot pointers and the first and last descriptor (cheap enough for every run)
  uint32_t mark = 2166136261u;
  auto mix = [&](const void* p, size_t n) {
    const unsigned char* b = static_cast<const unsigned char*>(p);
    for (size_t i = 0; i < n; ++i) { mark ^= b[i]; mark *= 16777619u; }
  };
  mix(&n_tds, sizeof n_tds); mix(&n_events, sizeof n_events); mix(&n_tensors, sizeof n_tensors);
  mix(&tds[0], sizeof(moe_tf_td)); mix(&tds[n_tds - 1], sizeof(moe_tf_td)); mix(slots, sizeof(void*) * (size_t)n_tensors);
  const int magic = (int)(mark | 1u);
  if (upload) {
    if (cudaMemcpyAsync(ws + sizeof(int) * TF_MAGIC, &magic, sizeof magic, cudaMemcpyHostToDevice, st) != cudaSuccess) return MOE_ERR_CUDA;   // the compiled plan is shape-stable: it is uploaded once and reused step after step (Section 4.3)
    if (cudaMemcpyAsync(ws + tf_slots_offset(n_events), slots, sizeof(void*) * (size_t)n_tensors, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return MOE_ERR_CUDA;
    if (cudaMemcpyAsync(ws + tf_tds_offset(n_events, n_tensors), tds, sizeof(moe_tf_td) * (size_t)n_tds, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return MOE_ERR_CUDA;
  }
  TfArgs a;
  a.tds = reinterpret_cast<const moe_tf_td*>(ws + tf_tds_offset(n_events, n_tensors));
  a.n_tds = n_tds;
  a.slots = reinterpret_cast<void* const*>(ws + tf_slots_offset(n_events));
  a.ws = reinterpret_cast<int*>(ws);
  a.magic = magic;
  a.budget_ns = 2000ull * 1000 * 1000;
  void* params[] = {&a};
  const int workers = TF_WORKERS_PER_SM * sms;
  const int grid = n_tds < workers ? n_tds : workers;
  const void* fn = reinterpret_cast<const void*>(taskflow_kernel);
  // cooperative: workers wait for one another's triggers, so all of them must be resident
  cudaError_t e = study_plain_launch().load() ? cudaLaunchKernel(fn, dim3(grid), dim3(STUDY_THREADS), params, 0, st)
                                              : cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(STUDY_THREADS), params, 0, st);
  return e == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

int moe_taskflow_status(const void* workspace, int32_t* status2, void* stream) {
  if (!workspace) return MOE_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return MOE_ERR_CUDA;
  int head[4];
  if (cudaMemcpy(head, workspace, sizeof head, cudaMemcpyDeviceToHost) != cudaSuccess) return MOE_ERR_CUDA;
  if (status2) { status2[0] = head[TF_STATUS]; status2[1] = head[TF_STATUS + 1]; }
  return MOE_OK;
}

}  // extern "C"
