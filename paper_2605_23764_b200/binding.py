"""ctypes binding of libmoe_b200.so: argument marshalling only.

Every function has the name and argument order of its C counterpart in include/moe_b200.h and
takes torch tensors where the C call takes pointers (CUDA tensors for device pointers, pinned
CPU tensors for the *_host calls).  The current torch stream is passed as the stream argument.
"""
from __future__ import annotations

import ctypes
import os

import torch

MOE_FLAG_RENORM_TOPK, MOE_FLAG_SAVE_FOR_BWD, MOE_FLAG_SERIAL_LAUNCH, MOE_FLAG_TRACE, MOE_FLAG_SIGMOID_GATE = 1, 2, 4, 8, 16
MOE_FLAG_DEFER_OUT_COPY = 32
MOE_BUF = {"counts": 0, "offsets": 1, "row_of": 2, "src_of": 3, "prow_of": 4, "pad_off": 5, "Xp": 6, "H": 7,
           "A": 8, "Y": 9, "dOutp": 10, "dH": 11, "dXp": 12, "meta": 13, "trace": 14, "event_counters": 15}
_BUF_DTYPE = {k: (torch.bfloat16 if k in ("Xp", "H", "A", "Y", "dOutp", "dH", "dXp") else torch.int32)
              for k in MOE_BUF}

EXPORTS = ["moe_workspace_bytes", "moe_create", "moe_destroy", "moe_route", "moe_layout", "moe_ffn_fwd",
           "moe_ffn_bwd", "moe_ffn_fwd_host", "moe_ffn_bwd_host", "moe_get_status", "moe_last_launch_count",
           "moe_set_wait_budget_ms", "moe_debug_buffer", "moe_strerror", "moe_last_cuda_error",
           "moe_set_profiling", "moe_get_phase_ms", "moe_route_host", "moe_layout_noalloc",
           "moe_debug_simulate_schedule", "moe_debug_set_unreachable_dependency", "moe_debug_trace", "moe_debug_set_plain_launch",
           "moe_sched_study_workspace_bytes", "moe_sched_study", "moe_sched_study_stats", "moe_router_fwd",
           "moe_router_bwd", "moe_taskflow_compile", "moe_taskflow_workspace_bytes", "moe_taskflow_run",
           "moe_taskflow_status", "moe_ep_plan", "moe_ep_dispatch", "moe_ep_combine"]
PHASES = ["route", "layout", "gather", "gemm_gate_up", "gemm_down", "combine", "bwd_gather", "act_grad",
          "dw_reduce", "wgrad_down", "gate_grad", "wgrad_gate_up", "bwd_combine", "fused_fwd", "fused_bwd"]


class MoeShape(ctypes.Structure):
    _fields_ = [("T_max", ctypes.c_int32), ("d", ctypes.c_int32), ("E", ctypes.c_int32), ("k", ctypes.c_int32),
                ("n_shared", ctypes.c_int32), ("F", ctypes.c_int32), ("flags", ctypes.c_uint32)]


class MoeError(RuntimeError):
    pass


MOE_TF_SWIGLU, MOE_TF_ADD, MOE_TF_NO_EVENT = 1, 2, 0xFFFFFFFF
MOE_EP_TILE_ROWS, MOE_EP_BLOCK_ROWS, MOE_EP_TOKEN_BLOCK = 32, 128, 32


class MoeEpPeer(ctypes.Structure):
    _fields_ = [("recv", ctypes.c_void_p), ("recv_meta", ctypes.c_void_p), ("recv_counters", ctypes.c_void_p),
                ("ret", ctypes.c_void_p), ("ret_counters", ctypes.c_void_p)]


class MoeEpTask(ctypes.Structure):
    _fields_ = [("expert", ctypes.c_int32), ("src_row0", ctypes.c_int32), ("nrows", ctypes.c_int32),
                ("dst_rank", ctypes.c_int32), ("dst_row0", ctypes.c_int32)]


class MoeEpLocal(ctypes.Structure):
    _fields_ = [("rank", ctypes.c_int32), ("T", ctypes.c_int32), ("n_tasks", ctypes.c_int32), ("recv_rows", ctypes.c_int32),
                ("x", ctypes.c_void_p), ("topk_w", ctypes.c_void_p), ("src_of", ctypes.c_void_p),
                ("tasks", ctypes.c_void_p), ("consumed", ctypes.c_void_p), ("ticket", ctypes.c_void_p)]


class MoeEpLocalCombine(ctypes.Structure):
    _fields_ = [("rank", ctypes.c_int32), ("T", ctypes.c_int32), ("recv_rows", ctypes.c_int32), ("pad", ctypes.c_int32),
                ("y", ctypes.c_void_p), ("out", ctypes.c_void_p), ("ticket", ctypes.c_void_p)]


class MoeTfTensor(ctypes.Structure):
    _fields_ = [("rows", ctypes.c_int32), ("cols", ctypes.c_int32)]


class MoeTfOperator(ctypes.Structure):
    _fields_ = [("op", ctypes.c_int32), ("n_inputs", ctypes.c_int32), ("inputs", ctypes.c_int32 * 4),
                ("n_outputs", ctypes.c_int32), ("outputs", ctypes.c_int32 * 2),
                ("n_split_inputs", ctypes.c_int32), ("split_input_idx", ctypes.c_int32 * 4),
                ("split_input_dim", ctypes.c_int32 * 4), ("split_output_dim", ctypes.c_int32 * 2),
                ("task_rows", ctypes.c_int32)]


class MoeTfTdesc(ctypes.Structure):
    _fields_ = [("slot", ctypes.c_uint32), ("row_offset", ctypes.c_uint32), ("rows", ctypes.c_uint32),
                ("cols", ctypes.c_uint32)]


class MoeTfTd(ctypes.Structure):
    _fields_ = [("task_type", ctypes.c_uint32), ("queue_type", ctypes.c_uint32), ("dependent_event", ctypes.c_uint32),
                ("dependent_threshold", ctypes.c_uint32), ("trigger_event", ctypes.c_uint32),
                ("task_index", ctypes.c_uint32), ("task_split_num", ctypes.c_uint32),
                ("task_split_value", ctypes.c_uint32), ("tiling_data_position", ctypes.c_uint32),
                ("n_inputs", ctypes.c_uint32), ("n_outputs", ctypes.c_uint32),
                ("inputs", MoeTfTdesc * 4), ("outputs", MoeTfTdesc * 2)]


_lib = None


def lib_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "libmoe_b200.so")


def load_library() -> ctypes.CDLL:
    """Load the C-ABI library; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise MoeError(f"{path} is missing: build it with `python -m paper_2605_23764_b200.build`")
    lib = ctypes.CDLL(path)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    lib.moe_workspace_bytes.restype = sz
    lib.moe_workspace_bytes.argtypes = [ctypes.POINTER(MoeShape)]
    lib.moe_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(MoeShape), vp, sz]
    lib.moe_destroy.argtypes = [vp]
    lib.moe_route.argtypes = [vp, vp, i32, vp, vp, vp, vp]
    lib.moe_layout.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp]
    lib.moe_ffn_fwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, vp]
    lib.moe_ffn_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp]
    lib.moe_ffn_fwd_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, vp]
    lib.moe_ffn_bwd_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, vp]
    lib.moe_get_status.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32)]
    lib.moe_last_launch_count.argtypes = [vp]
    lib.moe_set_wait_budget_ms.argtypes = [vp, i32]
    lib.moe_debug_buffer.argtypes = [vp, ctypes.c_int, ctypes.POINTER(vp), ctypes.POINTER(sz)]
    lib.moe_set_profiling.argtypes = [vp, i32]
    lib.moe_get_phase_ms.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    lib.moe_route_host.argtypes = [vp, vp, i32, vp, vp, vp]
    lib.moe_layout_noalloc.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp]
    lib.moe_debug_simulate_schedule.argtypes = [vp, i32, i32, i32, i32, i32, i32, i32, i32, i32, vp]
    lib.moe_debug_trace.argtypes = [vp, vp, sz, ctypes.POINTER(sz)]
    lib.moe_debug_set_unreachable_dependency.argtypes = [vp, i32]
    lib.moe_debug_set_plain_launch.argtypes = [vp, i32]
    lib.moe_router_fwd.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, vp]
    lib.moe_router_bwd.argtypes = [vp, vp, vp, vp, i32, vp, vp]
    lib.moe_taskflow_compile.argtypes = [ctypes.POINTER(MoeTfTensor), i32, ctypes.POINTER(MoeTfOperator), i32, i32,
                                         ctypes.POINTER(MoeTfTd), i32, ctypes.POINTER(i32), ctypes.POINTER(i32),
                                         ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32)]
    lib.moe_taskflow_workspace_bytes.restype = sz
    lib.moe_taskflow_workspace_bytes.argtypes = [i32, i32, i32]
    lib.moe_taskflow_run.argtypes = [ctypes.POINTER(MoeTfTd), i32, i32, ctypes.POINTER(vp), i32, vp, sz, i32, vp]
    lib.moe_taskflow_status.argtypes = [vp, ctypes.POINTER(i32), vp]
    lib.moe_ep_plan.argtypes = [ctypes.POINTER(i32), i32, i32, i32, ctypes.POINTER(MoeEpTask), i32, ctypes.POINTER(i32),
                                ctypes.POINTER(i32), ctypes.POINTER(i32)]
    lib.moe_ep_dispatch.argtypes = [ctypes.POINTER(MoeEpPeer), ctypes.POINTER(MoeEpLocal), i32, i32, i32, i32, vp, vp]
    lib.moe_ep_combine.argtypes = [ctypes.POINTER(MoeEpPeer), ctypes.POINTER(MoeEpLocalCombine), i32, i32, i32, i32, vp, vp]
    lib.moe_sched_study_workspace_bytes.restype = sz
    lib.moe_sched_study_workspace_bytes.argtypes = [i32, i32]
    lib.moe_sched_study.argtypes = [i32, vp, vp, vp, vp, i32, i32, i32, vp, sz, vp]
    lib.moe_sched_study_stats.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_uint64),
                                          ctypes.POINTER(ctypes.c_uint64), vp]
    lib.moe_strerror.restype = ctypes.c_char_p
    lib.moe_strerror.argtypes = [ctypes.c_int]
    lib.moe_last_cuda_error.restype = ctypes.c_char_p
    _lib = lib
    return lib


def _check(rc: int, what: str):
    if rc != 0:
        lib = load_library()
        msg = lib.moe_strerror(rc).decode()
        extra = lib.moe_last_cuda_error().decode()
        raise MoeError(f"{what}: {msg} ({rc})" + (f" [{extra}]" if extra and rc == -3 else ""))


def _dev(t, dtype, name):
    if t is None:
        return None
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise MoeError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return ctypes.c_void_p(t.data_ptr())


def _host(t, dtype, name):
    if t is None:
        return None
    if t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise MoeError(f"{name}: expected a contiguous CPU tensor of {dtype}")
    return ctypes.c_void_p(t.data_ptr())


_CTX_SHAPE = {}   # context handle -> (T_max, d, E, k, n_shared, F, flags): what the size checks need


def _shape_of(ctx):
    try:
        return _CTX_SHAPE[ctx.value]
    except (KeyError, AttributeError):
        raise MoeError("unknown context handle (not created by moe_create, or already destroyed)") from None


def _need(t, n, name):
    """An undersized tensor would make a kernel read or write out of bounds: refuse it here."""
    if t is not None and t.numel() < n:
        raise MoeError(f"{name}: {t.numel()} elements, the call needs {n}")


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _shape(T_max, d, E, k, n_shared, F, flags):
    return MoeShape(int(T_max), int(d), int(E), int(k), int(n_shared), int(F), int(flags))


def moe_strerror(code: int) -> str:
    return load_library().moe_strerror(code).decode()


def moe_workspace_bytes(T_max, d, E, k, n_shared, F, flags=0) -> int:
    s = _shape(T_max, d, E, k, n_shared, F, flags)
    return int(load_library().moe_workspace_bytes(ctypes.byref(s)))


def moe_create(T_max, d, E, k, n_shared, F, flags=0, workspace: torch.Tensor | None = None):
    """-> opaque context handle.  `workspace`: CUDA uint8 tensor (kept alive by the caller) or None."""
    s = _shape(T_max, d, E, k, n_shared, F, flags)
    h = ctypes.c_void_p()
    ws_ptr = ctypes.c_void_p(workspace.data_ptr()) if workspace is not None else None
    ws_bytes = workspace.numel() if workspace is not None else 0
    _check(load_library().moe_create(ctypes.byref(h), ctypes.byref(s), ws_ptr, ws_bytes), "moe_create")
    _CTX_SHAPE[h.value] = (int(T_max), int(d), int(E), int(k), int(n_shared), int(F), int(flags))
    return h


def moe_destroy(ctx):
    _check(load_library().moe_destroy(ctx), "moe_destroy")
    _CTX_SHAPE.pop(getattr(ctx, "value", None), None)


def moe_route(ctx, logits, T, topk_ids, topk_w, counts=None):
    _, _, E, k, _, _, _ = _shape_of(ctx)
    _need(logits, T * E, "logits"); _need(topk_ids, T * k, "topk_ids"); _need(topk_w, T * k, "topk_w")
    _need(counts, E, "counts")
    _check(load_library().moe_route(ctx, _dev(logits, torch.float32, "logits"), T,
                                    _dev(topk_ids, torch.int32, "topk_ids"), _dev(topk_w, torch.float32, "topk_w"),
                                    _dev(counts, torch.int32, "counts"), _stream()), "moe_route")


def moe_router_fwd(ctx, x, W_r, T, topk_ids, topk_w, logits=None, counts=None):
    _, d, E, k, _, _, _ = _shape_of(ctx)
    _need(x, T * d, "x"); _need(W_r, E * d, "W_r"); _need(topk_ids, T * k, "topk_ids"); _need(topk_w, T * k, "topk_w")
    _need(logits, T * E, "logits"); _need(counts, E, "counts")
    _check(load_library().moe_router_fwd(ctx, _dev(x, torch.bfloat16, "x"), _dev(W_r, torch.bfloat16, "W_r"), T,
                                         _dev(topk_ids, torch.int32, "topk_ids"), _dev(topk_w, torch.float32, "topk_w"),
                                         _dev(logits, torch.float32, "logits"), _dev(counts, torch.int32, "counts"),
                                         _stream()), "moe_router_fwd")


def moe_router_bwd(ctx, logits, topk_ids, d_topk_w, T, d_logits):
    _, _, E, k, _, _, _ = _shape_of(ctx)
    _need(logits, T * E, "logits"); _need(topk_ids, T * k, "topk_ids"); _need(d_topk_w, T * k, "d_topk_w")
    _need(d_logits, T * E, "d_logits")
    _check(load_library().moe_router_bwd(ctx, _dev(logits, torch.float32, "logits"), _dev(topk_ids, torch.int32, "topk_ids"),
                                         _dev(d_topk_w, torch.float32, "d_topk_w"), T,
                                         _dev(d_logits, torch.float32, "d_logits"), _stream()), "moe_router_bwd")


def moe_layout(ctx, topk_ids, T, counts=None, offsets=None, row_of=None, src_of=None):
    _, _, E, k, S, _, _ = _shape_of(ctx)
    _need(topk_ids, T * k, "topk_ids"); _need(counts, E + S, "counts"); _need(offsets, E + S + 1, "offsets")
    _need(row_of, T * (k + S), "row_of"); _need(src_of, T * (k + S), "src_of")
    _check(load_library().moe_layout(ctx, _dev(topk_ids, torch.int32, "topk_ids"), T,
                                     _dev(counts, torch.int32, "counts"), _dev(offsets, torch.int32, "offsets"),
                                     _dev(row_of, torch.int32, "row_of"), _dev(src_of, torch.int32, "src_of"),
                                     _stream()), "moe_layout")


def _need_layer_tensors(ctx, T, acts, ids_w, W_gate_up, W_down):
    _, d, E, k, S, F, _ = _shape_of(ctx)
    for name, t in acts.items():
        _need(t, T * d, name)
    for name, t in ids_w.items():
        _need(t, T * k, name)
    _need(W_gate_up, (E + S) * 2 * F * d, "W_gate_up")
    _need(W_down, (E + S) * d * F, "W_down")


def moe_ffn_fwd(ctx, x, topk_ids, topk_w, W_gate_up, W_down, out, T):
    bf = torch.bfloat16
    _need_layer_tensors(ctx, T, {"x": x, "out": out}, {"topk_ids": topk_ids, "topk_w": topk_w}, W_gate_up, W_down)
    _check(load_library().moe_ffn_fwd(ctx, _dev(x, bf, "x"), _dev(topk_ids, torch.int32, "topk_ids"),
                                      _dev(topk_w, torch.float32, "topk_w"), _dev(W_gate_up, bf, "W_gate_up"),
                                      _dev(W_down, bf, "W_down"), _dev(out, bf, "out"), T, _stream()), "moe_ffn_fwd")


def moe_ffn_bwd(ctx, dout, x, topk_ids, topk_w, W_gate_up, W_down, dx, dW_gate_up, dW_down, d_topk_w, T):
    bf = torch.bfloat16
    _need_layer_tensors(ctx, T, {"dout": dout, "x": x, "dx": dx},
                        {"topk_ids": topk_ids, "topk_w": topk_w, "d_topk_w": d_topk_w}, W_gate_up, W_down)
    _need(dW_gate_up, W_gate_up.numel(), "dW_gate_up"); _need(dW_down, W_down.numel(), "dW_down")
    _check(load_library().moe_ffn_bwd(ctx, _dev(dout, bf, "dout"), _dev(x, bf, "x"),
                                      _dev(topk_ids, torch.int32, "topk_ids"), _dev(topk_w, torch.float32, "topk_w"),
                                      _dev(W_gate_up, bf, "W_gate_up"), _dev(W_down, bf, "W_down"),
                                      _dev(dx, bf, "dx"), _dev(dW_gate_up, bf, "dW_gate_up"),
                                      _dev(dW_down, bf, "dW_down"), _dev(d_topk_w, torch.float32, "d_topk_w"),
                                      T, _stream()), "moe_ffn_bwd")


def moe_ffn_fwd_host(ctx, x_host, topk_ids_host, topk_w_host, W_gate_up, W_down, out_host, T):
    bf = torch.bfloat16
    _need_layer_tensors(ctx, T, {"x_host": x_host, "out_host": out_host},
                        {"topk_ids_host": topk_ids_host, "topk_w_host": topk_w_host}, W_gate_up, W_down)
    _check(load_library().moe_ffn_fwd_host(ctx, _host(x_host, bf, "x_host"),
                                           _host(topk_ids_host, torch.int32, "topk_ids_host"),
                                           _host(topk_w_host, torch.float32, "topk_w_host"),
                                           _dev(W_gate_up, bf, "W_gate_up"), _dev(W_down, bf, "W_down"),
                                           _host(out_host, bf, "out_host"), T, _stream()), "moe_ffn_fwd_host")


def moe_ffn_bwd_host(ctx, dout_host, W_gate_up, W_down, dx_host, dW_gate_up, dW_down, d_topk_w_host, T):
    bf = torch.bfloat16
    _need_layer_tensors(ctx, T, {"dout_host": dout_host, "dx_host": dx_host}, {"d_topk_w_host": d_topk_w_host},
                        W_gate_up, W_down)
    _need(dW_gate_up, W_gate_up.numel(), "dW_gate_up"); _need(dW_down, W_down.numel(), "dW_down")
    _check(load_library().moe_ffn_bwd_host(ctx, _host(dout_host, bf, "dout_host"), _dev(W_gate_up, bf, "W_gate_up"),
                                           _dev(W_down, bf, "W_down"), _host(dx_host, bf, "dx_host"),
                                           _dev(dW_gate_up, bf, "dW_gate_up"), _dev(dW_down, bf, "dW_down"),
                                           _host(d_topk_w_host, torch.float32, "d_topk_w_host"), T, _stream()),
           "moe_ffn_bwd_host")


def moe_get_status(ctx):
    code, detail = ctypes.c_int32(), ctypes.c_int32()
    _check(load_library().moe_get_status(ctx, ctypes.byref(code), ctypes.byref(detail)), "moe_get_status")
    return code.value, detail.value


def moe_last_launch_count(ctx) -> int:
    return int(load_library().moe_last_launch_count(ctx))


def moe_set_wait_budget_ms(ctx, ms: int):
    _check(load_library().moe_set_wait_budget_ms(ctx, ms), "moe_set_wait_budget_ms")


def moe_set_profiling(ctx, on: bool):
    _check(load_library().moe_set_profiling(ctx, 1 if on else 0), "moe_set_profiling")


def moe_get_phase_ms(ctx) -> dict:
    """Device milliseconds of each operator of the context's last call (operators it ran only)."""
    buf = (ctypes.c_float * len(PHASES))()
    _check(load_library().moe_get_phase_ms(ctx, buf), "moe_get_phase_ms")
    return {name: float(buf[i]) for i, name in enumerate(PHASES) if buf[i] > 0.0}


def moe_route_host(ctx, logits_host, T, topk_ids_host, topk_w_host):
    _, _, E, k, _, _, _ = _shape_of(ctx)
    _need(logits_host, T * E, "logits_host"); _need(topk_ids_host, T * k, "topk_ids_host")
    _need(topk_w_host, T * k, "topk_w_host")
    _check(load_library().moe_route_host(ctx, _host(logits_host, torch.float32, "logits_host"), T,
                                         _host(topk_ids_host, torch.int32, "topk_ids_host"),
                                         _host(topk_w_host, torch.float32, "topk_w_host"), _stream()),
           "moe_route_host")


def moe_layout_noalloc(topk_ids, T, E, k, n_shared, counts, offsets, row_of, src_of, status2=None):
    """Dispatch layout through the entry point that allocates nothing and needs no context (for
    callers that may not cudaMalloc).  All tensors are caller-owned CUDA int32 tensors."""
    i32 = torch.int32
    n, Ep = T * (k + n_shared), E + n_shared
    # a problem beyond the entry point's fixed limits is refused by the library itself before it touches memory
    if 0 <= n <= 262144 and Ep <= 1088 and -(-n // 2048) * Ep <= 131072:
        _need(topk_ids, T * k, "topk_ids"); _need(counts, Ep, "counts"); _need(offsets, Ep + 1, "offsets")
        _need(row_of, n, "row_of"); _need(src_of, n, "src_of"); _need(status2, 2, "status2")
    _check(load_library().moe_layout_noalloc(_dev(topk_ids, i32, "topk_ids"), T, E, k, n_shared,
                                             _dev(counts, i32, "counts"), _dev(offsets, i32, "offsets"),
                                             _dev(row_of, i32, "row_of"), _dev(src_of, i32, "src_of"),
                                             _dev(status2, i32, "status2"), _stream()), "moe_layout_noalloc")


MOE_STUDY_SERIAL, MOE_STUDY_STATIC, MOE_STUDY_DYNAMIC = 0, 1, 2


def moe_sched_study_workspace_bytes(M, tile_rows) -> int:
    return int(load_library().moe_sched_study_workspace_bytes(int(M), int(tile_rows)))


def moe_sched_study(mode, x, r, s, z, M, C, tile_rows, workspace):
    """SwiGLU + Add operator pair under one of the three schedules; all tensors are CUDA tensors
    (bf16 x[M][2C], r/s/z[M][C]; workspace: any dtype, at least moe_sched_study_workspace_bytes)."""
    bf = torch.bfloat16
    _need(x, M * 2 * C, "x"); _need(r, M * C, "r"); _need(s, M * C, "s"); _need(z, M * C, "z")
    if workspace is None or not workspace.is_cuda or not workspace.is_contiguous():
        raise MoeError("workspace: expected a contiguous CUDA tensor")
    nbytes = workspace.numel() * workspace.element_size()
    _check(load_library().moe_sched_study(int(mode), _dev(x, bf, "x"), _dev(r, bf, "r"), _dev(s, bf, "s"),
                                          _dev(z, bf, "z"), int(M), int(C), int(tile_rows),
                                          ctypes.c_void_p(workspace.data_ptr()), nbytes, _stream()), "moe_sched_study")


def moe_sched_study_stats(workspace):
    """((code, detail), dispatch_ns, tasks) of the last moe_sched_study call on this workspace."""
    st = (ctypes.c_int32 * 2)()
    ns, n = ctypes.c_uint64(0), ctypes.c_uint64(0)
    _check(load_library().moe_sched_study_stats(ctypes.c_void_p(workspace.data_ptr()), st, ctypes.byref(ns),
                                                ctypes.byref(n), _stream()), "moe_sched_study_stats")
    return (int(st[0]), int(st[1])), int(ns.value), int(n.value)


def tf_operator(op, inputs, outputs, task_rows, split_inputs=None, split_output_dims=None):
    """A graph node with its SplitSpec: split_inputs = None (partition origin) or [(input index, dim), ...]."""
    o = MoeTfOperator()
    o.op, o.n_inputs, o.n_outputs, o.task_rows = op, len(inputs), len(outputs), task_rows
    for i, t in enumerate(inputs):
        o.inputs[i] = t
    for j, t in enumerate(outputs):
        o.outputs[j] = t
        o.split_output_dim[j] = 0 if split_output_dims is None else split_output_dims[j]
    if split_inputs is None:
        o.n_split_inputs = -1
    else:
        o.n_split_inputs = len(split_inputs)
        for i, (idx, dim) in enumerate(split_inputs):
            o.split_input_idx[i], o.split_input_dim[i] = idx, dim
    return o


def moe_taskflow_compile(tensors, ops, lag_rows, td_cap=None):
    """tensors: [(rows, cols), ...]; ops: [MoeTfOperator, ...] -> dict(tds, n_tds, n_events, op_task_num,
    tensor_split_dim, tensor_split_num).  Host only."""
    ts = (MoeTfTensor * len(tensors))(*[MoeTfTensor(int(r), int(c)) for r, c in tensors])
    os_ = (MoeTfOperator * len(ops))(*ops)
    if td_cap is None:
        td_cap = sum(max(1, -(-tensors[o.outputs[0]][0] // max(1, o.task_rows))) for o in ops)
    tds = (MoeTfTd * max(1, td_cap))()
    n_tds, n_ev = ctypes.c_int32(0), ctypes.c_int32(0)
    tn = (ctypes.c_int32 * len(ops))()
    sd, sn = (ctypes.c_int32 * len(tensors))(), (ctypes.c_int32 * len(tensors))()
    _check(load_library().moe_taskflow_compile(ts, len(tensors), os_, len(ops), int(lag_rows), tds, td_cap,
                                               ctypes.byref(n_tds), ctypes.byref(n_ev), tn, sd, sn), "moe_taskflow_compile")
    return {"tds": tds, "n_tds": n_tds.value, "n_events": n_ev.value, "op_task_num": list(tn),
            "tensor_split_dim": list(sd), "tensor_split_num": list(sn)}


def moe_taskflow_workspace_bytes(n_tds, n_events, n_tensors) -> int:
    return int(load_library().moe_taskflow_workspace_bytes(int(n_tds), int(n_events), int(n_tensors)))


def moe_taskflow_run(plan, slots, shapes, workspace, upload=True):
    """Run a compiled plan: slots = one CUDA bf16 tensor per graph tensor, shapes = the (rows, cols) the plan was
    compiled for (each tensor must hold at least that many elements)."""
    for i, (t, (r, c)) in enumerate(zip(slots, shapes)):
        _need(t, r * c, f"slots[{i}]")
        _dev(t, torch.bfloat16, f"slots[{i}]")
    if len(slots) != len(shapes) or workspace is None or not workspace.is_cuda or not workspace.is_contiguous():
        raise MoeError("slots / workspace: expected one CUDA tensor per graph tensor and a contiguous CUDA workspace")
    ptrs = (ctypes.c_void_p * len(slots))(*[t.data_ptr() for t in slots])
    nbytes = workspace.numel() * workspace.element_size()
    _check(load_library().moe_taskflow_run(plan["tds"], plan["n_tds"], plan["n_events"], ptrs, len(slots),
                                           ctypes.c_void_p(workspace.data_ptr()), nbytes, 1 if upload else 0, _stream()),
           "moe_taskflow_run")


def moe_taskflow_status(workspace):
    st = (ctypes.c_int32 * 2)()
    _check(load_library().moe_taskflow_status(ctypes.c_void_p(workspace.data_ptr()), st, _stream()), "moe_taskflow_status")
    return int(st[0]), int(st[1])


def moe_ep_plan(counts, rank):
    """counts: int array [R][E] (every rank's per-expert row counts) -> (tasks [n][5] int32 numpy array: expert,
    src_row0, nrows, dst_rank, dst_row0; recv_rows [R]; recv_expert_offsets [E/R+1] of `rank`).  Host only."""
    import numpy as np
    c = np.ascontiguousarray(counts, dtype=np.int32)
    R, E = c.shape
    cap = (int(c[rank].sum()) if 0 <= rank < R else 0) // MOE_EP_TILE_ROWS + E + 1
    tasks = (MoeEpTask * cap)()
    n = ctypes.c_int32(0)
    rr = (ctypes.c_int32 * R)()
    off = (ctypes.c_int32 * (E // max(R, 1) + 1))()
    _check(load_library().moe_ep_plan(c.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), R, E, int(rank), tasks, cap,
                                      ctypes.byref(n), rr, off), "moe_ep_plan")
    arr = np.array([[t.expert, t.src_row0, t.nrows, t.dst_rank, t.dst_row0] for t in tasks[:n.value]],
                   dtype=np.int32).reshape(n.value, 5)
    return arr, np.array(list(rr), dtype=np.int32), np.array(list(off), dtype=np.int32)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def moe_ep_peer(recv, recv_meta, recv_counters, ret, ret_counters):
    """What one rank exposes: CUDA tensors (bf16 recv/ret, int32 meta/counters) living on, or peer-mapped into, the
    calling device."""
    return MoeEpPeer(_ptr(recv).value if recv is not None else None, _ptr(recv_meta).value if recv_meta is not None else None,
                     _ptr(recv_counters).value, _ptr(ret).value if ret is not None else None, _ptr(ret_counters).value)


def moe_ep_dispatch(peers, locals_, k, d, status):
    """peers: [MoeEpPeer] for every rank; locals_: [dict(rank, T, x, topk_w, src_of, tasks (CUDA int32 [n,5]), recv_rows,
    consumed|None, ticket)] for the ranks this call acts for; status: CUDA int32[4]."""
    R = len(peers)
    ps = (MoeEpPeer * R)(*peers)
    ls = (MoeEpLocal * len(locals_))()
    for i, l in enumerate(locals_):
        _need(l["x"], l["T"] * d, "x"); _need(l["topk_w"], l["T"] * k, "topk_w"); _need(l["src_of"], l["T"] * k, "src_of")
        _need(l.get("consumed"), l["recv_rows"] * d, "consumed"); _need(l["ticket"], 2, "ticket")
        n_tasks = 0 if l["tasks"] is None else l["tasks"].shape[0]
        ls[i] = MoeEpLocal(l["rank"], l["T"], n_tasks, l["recv_rows"], _ptr(l["x"]), _ptr(l["topk_w"]), _ptr(l["src_of"]),
                           _ptr(l["tasks"]), _ptr(l.get("consumed")), _ptr(l["ticket"]))
    _need(status, 4, "status")
    _check(load_library().moe_ep_dispatch(ps, ls, len(locals_), R, k, d, _dev(status, torch.int32, "status"), _stream()),
           "moe_ep_dispatch")


def moe_ep_combine(peers, locals_, k, d, status):
    """locals_: [dict(rank, T, recv_rows, y, out, ticket)]."""
    R = len(peers)
    ps = (MoeEpPeer * R)(*peers)
    ls = (MoeEpLocalCombine * len(locals_))()
    for i, l in enumerate(locals_):
        _need(l["y"], l["recv_rows"] * d, "y"); _need(l["out"], l["T"] * d, "out"); _need(l["ticket"], 2, "ticket")
        ls[i] = MoeEpLocalCombine(l["rank"], l["T"], l["recv_rows"], 0, _ptr(l["y"]), _ptr(l["out"]), _ptr(l["ticket"]))
    _need(status, 4, "status")
    _check(load_library().moe_ep_combine(ps, ls, len(locals_), R, k, d, _dev(status, torch.int32, "status"), _stream()),
           "moe_ep_combine")


def moe_debug_simulate_schedule(counts, T, k, n_shared, d, F, is_bwd, pairs, vec_workers):
    """Host-only schedule check; returns (code, stats) with code 0 = schedule is sound."""
    c = (ctypes.c_int32 * len(counts))(*[int(v) for v in counts])
    stats = (ctypes.c_int64 * 4)()
    rc = load_library().moe_debug_simulate_schedule(c, len(counts), T, k, n_shared, d, F, int(is_bwd), pairs,
                                                    vec_workers, stats)
    return rc, list(stats)


class MoeTraceRecord(ctypes.Structure):
    _fields_ = [("t0_ns", ctypes.c_uint64), ("t1_ns", ctypes.c_uint64), ("role", ctypes.c_uint8),
                ("phase", ctypes.c_uint8), ("pad", ctypes.c_uint16), ("item", ctypes.c_int32),
                ("cta", ctypes.c_uint32), ("dep_ns", ctypes.c_uint32)]


def moe_debug_trace(ctx, max_records=1 << 18):
    """-> (records as a list of dicts, number of records the launch produced)."""
    buf = (MoeTraceRecord * max_records)()
    n = ctypes.c_size_t()
    _check(load_library().moe_debug_trace(ctx, buf, max_records, ctypes.byref(n)), "moe_debug_trace")
    got = min(n.value, max_records)
    recs = [{"t0": r.t0_ns, "t1": r.t1_ns, "role": r.role, "phase": r.phase, "item": r.item, "cta": r.cta,
             "dep_ns": r.dep_ns} for r in buf[:got]]
    return recs, n.value


def moe_debug_set_unreachable_dependency(ctx, on: bool):
    _check(load_library().moe_debug_set_unreachable_dependency(ctx, 1 if on else 0),
           "moe_debug_set_unreachable_dependency")


def moe_debug_set_plain_launch(ctx, on: bool):
    _check(load_library().moe_debug_set_plain_launch(ctx, 1 if on else 0), "moe_debug_set_plain_launch")


class _DevView:
    """Minimal __cuda_array_interface__ holder so torch can view library-owned device memory."""

    def __init__(self, ptr, n, typestr):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": typestr, "data": (ptr, False), "version": 2}


def moe_debug_buffer(ctx, which: str) -> torch.Tensor:
    """Copy of a workspace tensor of the last call (see MOE_BUF_* in the header)."""
    ptr, n = ctypes.c_void_p(), ctypes.c_size_t()
    _check(load_library().moe_debug_buffer(ctx, MOE_BUF[which], ctypes.byref(ptr), ctypes.byref(n)),
           "moe_debug_buffer")
    if _BUF_DTYPE[which] == torch.int32:
        return torch.as_tensor(_DevView(ptr.value, n.value, "<i4"), device="cuda").clone()
    raw = torch.as_tensor(_DevView(ptr.value, n.value, "<i2"), device="cuda")
    return raw.view(torch.bfloat16).clone()


class MoeLayer:
    """Owns a context and its workspace (a torch allocation); allocates outputs; same calls as the C ABI."""

    def __init__(self, T_max, d, E, k, n_shared, F, renorm=False, save_for_bwd=False, serial=False, trace=False,
                 sigmoid_gate=False, defer_out_copy=False):
        self.T_max, self.d, self.E, self.k, self.S, self.F = T_max, d, E, k, n_shared, F
        self.flags = ((MOE_FLAG_RENORM_TOPK if renorm else 0) | (MOE_FLAG_SAVE_FOR_BWD if save_for_bwd else 0) |
                      (MOE_FLAG_SERIAL_LAUNCH if serial else 0) | (MOE_FLAG_TRACE if trace else 0) |
                      (MOE_FLAG_SIGMOID_GATE if sigmoid_gate else 0) | (MOE_FLAG_DEFER_OUT_COPY if defer_out_copy else 0))
        nbytes = moe_workspace_bytes(T_max, d, E, k, n_shared, F, self.flags)
        if nbytes == 0:
            raise MoeError("invalid shape")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        self.ctx = moe_create(T_max, d, E, k, n_shared, F, self.flags, self.workspace)

    def close(self):
        if self.ctx is not None:
            torch.cuda.synchronize()
            moe_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def route(self, logits, with_counts=False):
        T = logits.shape[0]
        ids = torch.empty(T, self.k, dtype=torch.int32, device="cuda")
        w = torch.empty(T, self.k, dtype=torch.float32, device="cuda")
        counts = torch.empty(self.E, dtype=torch.int32, device="cuda") if with_counts else None
        moe_route(self.ctx, logits, T, ids, w, counts)
        return (ids, w, counts) if with_counts else (ids, w)

    def layout(self, topk_ids):
        T = topk_ids.shape[0]
        n, Ep = T * (self.k + self.S), self.E + self.S
        i32 = dict(dtype=torch.int32, device="cuda")
        counts, offsets = torch.empty(Ep, **i32), torch.empty(Ep + 1, **i32)
        row_of, src_of = torch.empty(n, **i32), torch.empty(n, **i32)
        moe_layout(self.ctx, topk_ids, T, counts, offsets, row_of, src_of)
        return counts, offsets, row_of, src_of

    def ffn_fwd(self, x, topk_ids, topk_w, W_gate_up, W_down, out=None):
        T = x.shape[0]
        if out is None:
            out = torch.empty(T, self.d, dtype=torch.bfloat16, device="cuda")
        moe_ffn_fwd(self.ctx, x, topk_ids, topk_w, W_gate_up, W_down, out, T)
        return out

    def ffn_bwd(self, dout, x, topk_ids, topk_w, W_gate_up, W_down, dx=None, dW_gate_up=None, dW_down=None,
                d_topk_w=None, want_d_topk_w=True):
        T = x.shape[0]
        dx = torch.empty_like(x) if dx is None else dx
        dW_gate_up = torch.empty_like(W_gate_up) if dW_gate_up is None else dW_gate_up
        dW_down = torch.empty_like(W_down) if dW_down is None else dW_down
        if d_topk_w is None and want_d_topk_w:
            d_topk_w = torch.empty(T, self.k, dtype=torch.float32, device="cuda")
        moe_ffn_bwd(self.ctx, dout, x, topk_ids, topk_w, W_gate_up, W_down, dx, dW_gate_up, dW_down, d_topk_w, T)
        return dx, dW_gate_up, dW_down, d_topk_w

    def status(self):
        return moe_get_status(self.ctx)

    def launches(self):
        return moe_last_launch_count(self.ctx)

    def debug(self, which):
        return moe_debug_buffer(self.ctx, which)
