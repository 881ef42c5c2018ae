#!/usr/bin/env python
"""Benchmark of the Dispatch->Combine MoE-FFN layer on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--impl reference]

One step = one pass of the whole hot path on one batch of seeded synthetic input: routing,
forward (dispatch layout, permute-gather, grouped GEMM gate+up with SwiGLU, grouped GEMM down,
combine) and, for the training workload, backward (the seven backward operators).  Rank 0
prints ONE JSON line.  Throughput counts 6*R*d*F FLOP per forward and 12*R*d*F per backward
(R = tokens x experts per token).

The headline `value` is the library's default launch mode: one persistent dependency-driven
launch per pass.  The one-launch-per-operator mode is timed in the same run and reported as
`other_launch_mode`; `all_configs` holds both modes for the forward-only workloads;
`scheduling_study` holds the SwiGLU+Add scheduling microbenchmark (Section 6): serial, statically
interleaved and dynamically dispatched, with the dispatch time per task; `router_in_path` the router GEMM +
top-k launch on the workload's shape (it is outside the timed step, whose routing starts from given logits).
With N > 1 every rank runs an independent replica on its own GPU (the layer is not sharded;
there is no data-path collective); `python bench.py --gpus N` without a launcher starts the N
ranks itself.
"""
from __future__ import annotations

import argparse
import gc
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import configs  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
METRIC = "moe_ffn_dispatch_to_combine_tflops"
LAUNCH_NAMES = {"serial": "serial kernels (one launch per operator)",
                "fused": "fused persistent (one launch each for forward and backward, after the index-only "
                         "layout kernels)"}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


# ----------------------------------------------------------------------------------------------
# algorithmic work per operator (what the method must compute / move: inputs read once, outputs
# written once; padding rows and re-reads are not credited)
# ----------------------------------------------------------------------------------------------
def phase_work(cfg, train):
    R, d, F, Ep, T = cfg.R, cfg.d, cfg.F, cfg.Ep, cfg.T
    bf = 2
    W1, W2 = Ep * 2 * F * d * bf, Ep * d * F * bf
    work = {
        "gather": (0.0, T * d * bf + R * d * bf),
        "gemm_gate_up": (2.0 * R * d * 2 * F, R * d * bf + W1 + R * F * bf + (R * 2 * F * bf if train else 0)),
        "gemm_down": (2.0 * R * F * d, R * F * bf + W2 + R * d * bf),
        "combine": (0.0, R * d * bf + T * d * bf),
    }
    work["fused_fwd"] = (6.0 * R * d * F, W1 + W2 + 2 * T * d * bf + (R * 2 * F * bf if train else 0))
    if train:
        # backward alone: weights read once, weight gradients written once, dout in, dx out, saved pre-activations in
        work["fused_bwd"] = (12.0 * R * d * F, 2 * (W1 + W2) + 3 * T * d * bf + R * 2 * F * bf)
        work.update({
            "bwd_gather": (0.0, T * d * bf + R * d * bf),
            "act_grad": (2.0 * R * d * F, R * d * bf + W2 + R * 2 * F * bf * 2),
            "wgrad_down": (2.0 * R * d * F, R * d * bf + R * F * bf + W2),
            "gate_grad": (2.0 * R * 2 * F * d, R * 2 * F * bf + W1 + R * d * bf),
            "wgrad_gate_up": (2.0 * R * 2 * F * d, R * 2 * F * bf + R * d * bf + W1),
            "bwd_combine": (0.0, R * d * bf + T * d * bf),
        })
    return work


def step_flops(cfg, train):
    return cfg.flops_fwd() * (3.0 if train else 1.0)


def step_min_bytes(cfg, train):
    """Minimum HBM traffic of a step: weights, activations in and out, weight gradients."""
    bf = 2
    W = cfg.weight_bytes()
    io = 2 * cfg.T * cfg.d * bf
    if not train:
        return W + io
    saved = 2 * cfg.R * 2 * cfg.F * bf  # pre-activations written by forward, read by backward
    return 3 * W + 2 * io + cfg.T * cfg.d * bf + saved


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def dist_setup():
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    return world, rank, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()


def max_over_ranks(v, world, device="cuda"):
    """The slowest rank's time: replicas are independent, the job is as slow as its slowest one."""
    if world == 1:
        return v
    import torch.distributed as dist
    t = torch.tensor([v], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(local_ms_per_step, flops_per_replica_step, world, device="cuda"):
    """Whole-job TFLOP/s of `world` independent replicas (weak scaling): all ranks' work over the
    slowest rank's time."""
    ms = max_over_ranks(local_ms_per_step, world, device)
    return world * flops_per_replica_step / (ms * 1e-3) / 1e12, ms


# ----------------------------------------------------------------------------------------------
# CPU oracle legs (rank 0 only): a bounded sample of the same workload
# ----------------------------------------------------------------------------------------------
def oracle_sample(cfg, train, n_experts, rows_per_expert, inputs=None):
    """Times the oracle on an exact sub-problem of the workload: up to `rows_per_expert` rows of each
    of `n_experts` median-loaded experts, ONE oracle call over all of them (forward, and backward if
    `train`), so that its loops over tokens and over experts have work for every thread.

    Returns (seconds, flops, description).  An expert's rows and weight gradient need only that
    expert's slabs, which is what makes the sample exact."""
    import oracle
    dev = "cpu"
    x = inputs["x"].cpu() if inputs else configs.make_x(cfg, dev)
    logits = inputs["logits"].cpu() if inputs else configs.make_logits(cfg, x)
    ids, w = oracle.route(logits, cfg.k, cfg.renorm)
    ids_t, w_t = torch.from_numpy(ids), torch.from_numpy(w)
    dout = (inputs["dout"].cpu() if inputs else configs.make_dout(cfg, dev)) if train else None
    counts = torch.bincount(ids_t.flatten().long(), minlength=cfg.E)
    order = torch.argsort(counts, descending=True)
    lo = max(0, len(order) // 2 - n_experts // 2)
    picked = [int(e) for e in order[lo: lo + n_experts] if counts[int(e)] > 0]
    toks, sub_ids, sub_w = [], [], []
    for i, e in enumerate(picked):
        tok, slot = torch.nonzero(ids_t == e, as_tuple=True)
        tok, slot = tok[:rows_per_expert], slot[:rows_per_expert]
        toks.append(tok)
        sub_ids.append(torch.full((tok.numel(), 1), i, dtype=torch.int32))
        sub_w.append(w_t[tok, slot][:, None])
    tok = torch.cat(toks)
    sub_ids, sub_w = torch.cat(sub_ids), torch.cat(sub_w)
    W1 = torch.stack([configs.w_gate_up_slab(cfg, e) for e in picked])
    W2 = torch.stack([configs.w_down_slab(cfg, e) for e in picked])
    xs = x[tok]
    rows = tok.numel()
    t0 = time.perf_counter()
    oracle.fwd(xs, sub_ids, sub_w, W1, W2)
    if train:
        oracle.bwd(dout[tok], xs, sub_ids, sub_w, W1, W2)
    secs = time.perf_counter() - t0
    flops = 6.0 * rows * cfg.d * cfg.F * (3.0 if train else 1.0)
    desc = (f"{'fwd+bwd' if train else 'fwd'} of {rows} rows of {len(picked)} median-loaded experts in one oracle "
            f"call (of {cfg.R} rows, {cfg.Ep} experts)")
    return secs, flops, desc


def calibrate_sample(cfg, train, threads, target_s=15.0):
    """(experts, rows per expert) giving roughly `target_s` seconds of oracle work with every thread
    busy: at least `threads` experts, as many rows each as the time allows.  The rate is a fixed estimate
    of the plain-loop fp64 oracle per thread, not a measurement."""
    n_exp = int(min(cfg.E, max(threads, 1)))
    flop_per_row = 6.0 * cfg.d * cfg.F * (3.0 if train else 1.0)
    est_rate_per_thread = 0.15e9 if train else 0.5e9
    rows = max(1, int(target_s * est_rate_per_thread * min(threads, n_exp) / flop_per_row))
    return n_exp, max(1, rows // n_exp)


def run_reference(args, cfg, train):
    import oracle
    n_exp, rows = calibrate_sample(cfg, train, oracle.threads(), target_s=4.0)
    times, flops, desc = [], 0.0, ""
    for i in range(args.warmup + args.steps):
        secs, flops, desc = oracle_sample(cfg, train, n_exp, rows)
        if i >= args.warmup:
            times.append(secs)
    ms = 1e3 * sum(times) / len(times)
    val = flops / (ms * 1e-3) / 1e12
    cfg_desc = workload_desc(cfg, train)
    cfg_desc["launch"] = "none (CPU oracle on host cores)"
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": cfg_desc, "gpu_launches": 0,
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": oracle.threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def workload_desc(cfg, train):
    return {"workload": cfg.name, "T": cfg.T, "d": cfg.d, "E": cfg.E, "top_k": cfg.k, "shared": cfg.S, "F": cfg.F,
            "pass": "route+fwd+bwd" if train else "route+fwd",
            "l2": "weights and expert-ordered activations exceed the 126 MB L2 (no flush needed)"
            if cfg.weight_bytes() > 4e8 else "L2 flushed between timed steps"}


# ----------------------------------------------------------------------------------------------
# one workload resident on the GPU, timed in one or both launch modes
# ----------------------------------------------------------------------------------------------
class Workload:
    def __init__(self, cfg, train):
        self.cfg, self.train = cfg, train
        self.inp = configs.make_inputs(cfg, "cuda")
        T = cfg.T
        self.ids = torch.empty(T, cfg.k, dtype=torch.int32, device="cuda")
        self.w = torch.empty(T, cfg.k, dtype=torch.float32, device="cuda")
        self.out = torch.empty_like(self.inp["x"])
        if train:
            self.dx = torch.empty_like(self.inp["x"])
            self.dW1, self.dW2 = torch.empty_like(self.inp["W_gate_up"]), torch.empty_like(self.inp["W_down"])
            self.dw = torch.empty(T, cfg.k, dtype=torch.float32, device="cuda")
        # weights that fit L2 would stay there from step to step: flush between timed steps
        self.flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if cfg.weight_bytes() <= 4e8 else None

    plain_launch = False   # --plain-launch: persistent launches without the cooperative attribute (profiler captures)

    def make_layer(self, mode, defer_out_copy=False):
        from paper_2605_23764_b200 import MoeLayer, binding as B
        c = self.cfg
        lay = MoeLayer(c.T, c.d, c.E, c.k, c.S, c.F, renorm=c.renorm, save_for_bwd=self.train, serial=(mode == "serial"),
                       defer_out_copy=defer_out_copy)
        if Workload.plain_launch:
            B.moe_debug_set_plain_launch(lay.ctx, True)
        return lay

    def step(self, lay, phases=None):
        """One pass of the hot path through the C ABI (device buffers).  -> kernels launched"""
        from paper_2605_23764_b200 import binding as B
        i, T, n = self.inp, self.cfg.T, 0
        B.moe_route(lay.ctx, i["logits"], T, self.ids, self.w)
        n += lay.launches()
        if phases is not None:
            phases.update(B.moe_get_phase_ms(lay.ctx))
        B.moe_ffn_fwd(lay.ctx, i["x"], self.ids, self.w, i["W_gate_up"], i["W_down"], self.out, T)
        n += lay.launches()
        if phases is not None:
            phases.update(B.moe_get_phase_ms(lay.ctx))
        if self.train:
            B.moe_ffn_bwd(lay.ctx, i["dout"], i["x"], self.ids, self.w, i["W_gate_up"], i["W_down"], self.dx, self.dW1,
                          self.dW2, self.dw, T)
            n += lay.launches()
            if phases is not None:
                phases.update(B.moe_get_phase_ms(lay.ctx))
        return n

    def measure(self, lay, steps, warmup, world, local, min_timed_ms=0.0):
        """W warm-up steps, then K timed steps back to back (CUDA events on the launching stream; the
        per-operator events inside the library are read after each call).  -> dict"""
        from paper_2605_23764_b200 import binding as B
        for _ in range(warmup - 1):
            self.step(lay)
        w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        w0.record(); self.step(lay); w1.record()
        torch.cuda.synchronize()
        assert lay.status() == (0, 0), "device-side error during warm-up"
        # The per-operator events are recorded in every timed step; READING them synchronises the stream, which
        # a sub-millisecond step would feel: short steps are read every few steps only (about one read per 5 ms).
        if min_timed_ms:   # short workloads: enough steps for a timed region as long as the headline workload's
            steps = max(steps, min(4000, int(min_timed_ms / max(w0.elapsed_time(w1), 1e-3)) + 1))
        read_every = max(1, min(steps, int(5.0 / max(w0.elapsed_time(w1), 1e-3))))
        B.moe_set_profiling(lay.ctx, True)
        phase_sum, n_launch, n_reads = {}, 0, 0
        sampler = ClockSampler(local)
        sampler.start()
        barrier(world)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        flush_ms, flush_events = 0.0, []
        ev0.record()
        for i in range(steps):
            if self.flush is not None:
                f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                f0.record(); self.flush.zero_(); f1.record()
                flush_events.append((f0, f1))
            read = (i % read_every) == read_every - 1
            ph = {} if read else None
            n_launch += self.step(lay, phases=ph)
            if read:
                n_reads += 1
                for kname, v in ph.items():
                    phase_sum[kname] = phase_sum.get(kname, 0.0) + v
        ev1.record()
        barrier(world)
        clk = sampler.stop()
        for f0, f1 in flush_events:
            flush_ms += f0.elapsed_time(f1)
        local_ms = (ev0.elapsed_time(ev1) - flush_ms) / steps
        value_all, ms = replica_throughput(local_ms, step_flops(self.cfg, self.train), world)
        B.moe_set_profiling(lay.ctx, False)
        code, detail = lay.status()
        assert code == 0, f"device-side error {code} detail {detail:#x}"
        return {"ms_per_step": ms, "value": value_all,
                "phases_ms": {k: v / max(1, n_reads) for k, v in phase_sum.items()}, "launches": n_launch,
                "clocks": clk, "timed_ms": ms * steps, "steps": steps}


def rooflines(cfg, train, res, peaks):
    """Roofline of the operator with the largest time, and of the whole step."""
    work = phase_work(cfg, train)
    phases_ms = res["phases_ms"]
    # sustained peak for work timed inside a long, power-capped region (the clocks sampled during the timed
    # steps say which): more than 0.5 s of timed work, or the power cap active with SM clocks a fifth or
    # more below their maximum; burst peak otherwise
    clk = res.get("clocks") or {}
    capped = ("sw_power_cap" in (clk.get("reasons") or []) and clk.get("sm_mhz") and clk.get("sm_max_mhz")
              and clk["sm_mhz"] < 0.8 * clk["sm_max_mhz"])
    sustained = res["timed_ms"] > 500 or capped
    peak_tf = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    peak_gb = peaks["hbm_gbs"]
    dom = max((k for k in phases_ms if k in work), key=lambda k: phases_ms[k], default=None)
    roof = None
    if dom:
        fl, by = work[dom]
        t_s = phases_ms[dom] * 1e-3
        tensor_bound = fl / (peak_tf * 1e12) >= by / (peak_gb * 1e9)
        if tensor_bound:
            roof = {"kernel": dom, "bound": "tensor", "achieved": fl / t_s / 1e12, "peak": peak_tf, "unit": "TFLOP/s"}
        else:
            roof = {"kernel": dom, "bound": "hbm", "achieved": by / t_s / 1e9, "peak": peak_gb, "unit": "GB/s"}
        roof["frac"] = roof["achieved"] / roof["peak"]
        roof["peak_source"] = peaks["source"] + ((" sustained" if sustained else " burst") if tensor_bound else "")
        roof["traffic"] = ncu_traffic(dom, cfg)
        roof["launch_ms"] = phases_ms[dom]
    flops = step_flops(cfg, train)
    flop_ms = flops / (peak_tf * 1e12) * 1e3
    hbm_ms = step_min_bytes(cfg, train) / (peak_gb * 1e9) * 1e3
    t_roof = max(flop_ms, hbm_ms)
    step_roof = {"roofline_ms": t_roof, "frac": t_roof / res["ms_per_step"], "flop_ms": flop_ms, "hbm_ms": hbm_ms,
                 "bound": "tensor" if flop_ms >= hbm_ms else "hbm",
                 "tensor_peak": "sustained" if sustained else "burst"}
    return roof, step_roof


def ncu_traffic(phase, cfg):
    """DRAM bytes per launch of `phase` on this workload from the committed ncu summary, if any."""
    path = os.path.join(ROOT, "profiles", "ncu_dram_traffic.txt")
    if not os.path.exists(path):
        return None
    for ln in open(path):
        parts = ln.split()
        if len(parts) >= 3 and not ln.startswith("#") and parts[0] == phase and parts[1] == cfg.name:
            return float(parts[2])
    return None


def run_e2e(wl, layer, steps, world):
    """The same step through the host-buffer entry points: pinned host inputs in, results out, copies timed."""
    from paper_2605_23764_b200 import binding as B
    cfg, train, inp = wl.cfg, wl.train, wl.inp
    T = cfg.T
    pin = dict(pin_memory=True)
    xh, lh = inp["x"].cpu().pin_memory(), inp["logits"].cpu().pin_memory()
    idh = torch.empty(T, cfg.k, dtype=torch.int32, **pin)
    wh = torch.empty(T, cfg.k, dtype=torch.float32, **pin)
    oh = torch.empty(T, cfg.d, dtype=torch.bfloat16, **pin)
    h2d = lh.numel() * 4 + xh.numel() * 2 + idh.numel() * 4 + wh.numel() * 4
    d2h = idh.numel() * 4 + wh.numel() * 4 + oh.numel() * 2
    if train:
        doh = inp["dout"].cpu().pin_memory()
        dxh = torch.empty(T, cfg.d, dtype=torch.bfloat16, **pin)
        dwh = torch.empty(T, cfg.k, dtype=torch.float32, **pin)
        h2d += doh.numel() * 2
        d2h += dxh.numel() * 2 + dwh.numel() * 4

    def e2e_step():
        B.moe_route_host(layer.ctx, lh, T, idh, wh)
        B.moe_ffn_fwd_host(layer.ctx, xh, idh, wh, inp["W_gate_up"], inp["W_down"], oh, T)
        if train:
            B.moe_ffn_bwd_host(layer.ctx, doh, inp["W_gate_up"], inp["W_down"], dxh, wl.dW1, wl.dW2, dwh, T)

    for _ in range(2):
        e2e_step()
    barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        e2e_step()
    e1.record()
    barrier(world)
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), world) / steps
    assert layer.status()[0] == 0
    assert torch.equal(oh.cuda(), wl.out), "host-buffer path disagrees with the device-buffer path"
    return {"value": world * step_flops(cfg, train) / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}


def scheduling_study(peaks, iters=30):
    """SwiGLU(M x 4096) + Add(M x 2048) under the three schedules (Section 6.1, 6.2): median microseconds per
    pass with L2 flushed before each, and the workers' dispatch time per task."""
    from paper_2605_23764_b200 import binding as B
    dev, C, tile_rows = torch.device("cuda"), 2048, 8
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    rows = []
    for M in (2048, 8192, 32768):
        g = torch.Generator(device="cuda").manual_seed(1000 + M)
        x = torch.randn(M, 2 * C, device=dev, generator=g).to(torch.bfloat16)
        r = torch.randn(M, C, device=dev, generator=g).to(torch.bfloat16)
        s, z = torch.empty_like(r), torch.empty_like(r)
        ws = torch.empty(B.moe_sched_study_workspace_bytes(M, tile_rows), dtype=torch.uint8, device=dev)
        algo_bytes = M * C * 2 * (2 + 1 + 1 + 1 + 1)   # x (2C), s written and read, r, z: per row and column 2 bytes each
        row = {"M": M, "tile_rows": tile_rows, "tasks": 2 * (-(-M // tile_rows))}
        for mode, name in ((0, "serial"), (1, "static"), (2, "dynamic")):
            ts = []
            for it in range(iters + 3):
                flush.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); B.moe_sched_study(mode, x, r, s, z, M, C, tile_rows, ws); e1.record()
                torch.cuda.synchronize()
                if it >= 3:
                    ts.append(e0.elapsed_time(e1) * 1e3)
            status, ns, n = B.moe_sched_study_stats(ws)
            if status != (0, 0):
                raise SystemExit(f"scheduling study: device status {status}")
            us = sorted(ts)[len(ts) // 2]
            row[name] = {"us": us, "GBps": algo_bytes / us / 1e3, "frac_of_hbm_peak": algo_bytes / us / 1e3 / peaks["hbm_gbs"],
                         "dispatch_ns_per_task": (ns / n) if n else None}
        # the same pair compiled by the generic front end into task descriptors and run by the descriptor runtime
        shapes = [(M, 2 * C), (M, C), (M, C), (M, C)]
        plan = B.moe_taskflow_compile(shapes, [B.tf_operator(B.MOE_TF_SWIGLU, [0], [1], tile_rows, split_inputs=None),
                                               B.tf_operator(B.MOE_TF_ADD, [1, 2], [3], tile_rows, split_inputs=[(0, 0)])],
                                      lag_rows=tile_rows * 4 * torch.cuda.get_device_properties(0).multi_processor_count)
        tws = torch.empty(B.moe_taskflow_workspace_bytes(plan["n_tds"], plan["n_events"], 4), dtype=torch.uint8, device=dev)
        ts = []
        for it in range(iters + 3):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); B.moe_taskflow_run(plan, [x, s, r, z], shapes, tws, upload=(it == 0)); e1.record()
            torch.cuda.synchronize()
            if it >= 3:
                ts.append(e0.elapsed_time(e1) * 1e3)
        if B.moe_taskflow_status(tws) != (0, 0):
            raise SystemExit("taskflow runtime: device status")
        us = sorted(ts)[len(ts) // 2]
        row["descriptors"] = {"us": us, "GBps": algo_bytes / us / 1e3, "frac_of_hbm_peak": algo_bytes / us / 1e3 / peaks["hbm_gbs"],
                              "tasks": plan["n_tds"], "note": "descriptor table uploaded once, before the timed calls"}
        rows.append(row)
    return {"operators": "SwiGLU(M x 4096) -> s(M x 2048, bf16, in global memory) -> Add(M x 2048)",
            "timing": "CUDA events around each call (workspace clear + kernels), L2 flushed before each; median of %d" % iters,
            "rows": rows}


def router_in_path(cfg, peaks, iters=30):
    """The in-path router on the workload's shape: x W_r^T + softmax top-k in one launch (`moe_router_fwd`), and the
    score gradient (`moe_router_bwd`); median microseconds with L2 flushed before each call."""
    from paper_2605_23764_b200 import MoeLayer, binding as B
    dev = torch.device("cuda")
    T, d, E, k = cfg.T, cfg.d, cfg.E, cfg.k
    g = torch.Generator(device="cuda").manual_seed(77)
    x = torch.randn(T, d, device=dev, generator=g).to(torch.bfloat16)
    W = (torch.randn(E, d, device=dev, generator=g) * 0.02).to(torch.bfloat16)
    lay = MoeLayer(T, d, E, k, 0, 128, renorm=cfg.renorm)
    ids = torch.empty(T, k, dtype=torch.int32, device=dev)
    w = torch.empty(T, k, dtype=torch.float32, device=dev)
    logits = torch.empty(T, E, dtype=torch.float32, device=dev)
    dl = torch.empty_like(logits)
    gw = torch.randn(T, k, device=dev, generator=g)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def med(fn):
        ts = []
        for it in range(iters + 3):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            torch.cuda.synchronize()
            if it >= 3:
                ts.append(e0.elapsed_time(e1) * 1e3)
        return sorted(ts)[len(ts) // 2]

    us_f = med(lambda: B.moe_router_fwd(lay.ctx, x, W, T, ids, w, logits))
    us_b = med(lambda: B.moe_router_bwd(lay.ctx, logits, ids, gw, T, dl))
    assert lay.status() == (0, 0)
    lay.close()
    flop, by = 2.0 * T * d * E, 2.0 * T * d + 2.0 * E * d + 4.0 * T * E + 8.0 * T * k
    roof_us = max(flop / (peaks["bf16_tflops"] * 1e12), by / (peaks["hbm_gbs"] * 1e9)) * 1e6
    by_b = 2 * 4.0 * T * E + 8.0 * T * k
    return {"shape": {"T": T, "d": d, "E": E, "k": k},
            "fwd": {"us": us_f, "TFLOPs": flop / us_f / 1e6, "GBps": by / us_f / 1e3, "roofline_us": roof_us,
                    "frac": roof_us / us_f, "bound": "tensor" if flop / (peaks["bf16_tflops"] * 1e12) >= by / (peaks["hbm_gbs"] * 1e9) else "hbm"},
            "bwd": {"us": us_b, "GBps": by_b / us_b / 1e3, "frac": by_b / us_b / 1e3 / peaks["hbm_gbs"], "bound": "hbm"},
            "timing": "CUDA events around each call, L2 flushed before each; median of %d" % iters}


def ep_emulated(cfg, peaks, R=8, iters=20):
    """Expert-parallel Dispatch and Combine with one-sided put + signal (Section 4.1), the R ranks emulated on this one
    GPU (all buffers local, one cooperative launch plays every rank): the workload's tokens split evenly over the ranks.
    What is timed is the kernels' data path against local HBM; no NVLink is crossed."""
    import numpy as np
    from paper_2605_23764_b200 import MoeLayer, binding as B
    dev = torch.device("cuda")
    d, E, k = cfg.d, cfg.E, cfg.k
    if E % R or cfg.T % R:
        return None
    Tr = cfg.T // R
    g = torch.Generator(device="cuda").manual_seed(5)
    i32 = dict(dtype=torch.int32, device=dev)
    xs, ws, src, counts = [], [], [], []
    lay = MoeLayer(Tr, d, E, k, 0, 128, renorm=True)
    for s_ in range(R):
        x = torch.randn(Tr, d, device=dev, generator=g).to(torch.bfloat16)
        ids, w = lay.route(torch.randn(Tr, E, device=dev, generator=g))
        c = torch.empty(E, **i32); o = torch.empty(E + 1, **i32); ro = torch.empty(Tr * k, **i32); so = torch.empty(Tr * k, **i32)
        B.moe_layout(lay.ctx, ids, Tr, c, o, ro, so)
        torch.cuda.synchronize()
        xs.append(x); ws.append(w.clone()); src.append(so.clone()); counts.append(c.cpu().numpy())
    lay.close()
    counts = np.stack(counts).astype(np.int32)
    plans = [B.moe_ep_plan(counts, s_) for s_ in range(R)]
    rr = [int(v) for v in plans[0][1]]
    recv = [torch.empty(n, d, dtype=torch.bfloat16, device=dev) for n in rr]
    meta = [torch.empty(n, 4, **i32) for n in rr]
    rcnt = [torch.zeros(-(-n // B.MOE_EP_BLOCK_ROWS), **i32) for n in rr]
    ret = [torch.empty(Tr * k, d, dtype=torch.bfloat16, device=dev) for _ in range(R)]
    tcnt = [torch.zeros(-(-Tr // B.MOE_EP_TOKEN_BLOCK), **i32) for _ in range(R)]
    peers = [B.moe_ep_peer(recv[q], meta[q], rcnt[q], ret[q], tcnt[q]) for q in range(R)]
    tick = [torch.zeros(2, **i32) for _ in range(R)]
    tasks = [torch.from_numpy(plans[s_][0]).to(dev) for s_ in range(R)]
    out = [torch.empty(Tr, d, dtype=torch.bfloat16, device=dev) for _ in range(R)]
    status = torch.zeros(4, **i32)
    loc_d = [dict(rank=s_, T=Tr, x=xs[s_], topk_w=ws[s_], src_of=src[s_], tasks=tasks[s_], recv_rows=rr[s_], consumed=None,
                  ticket=tick[s_]) for s_ in range(R)]
    loc_c = [dict(rank=s_, T=Tr, recv_rows=rr[s_], y=recv[s_], out=out[s_], ticket=tick[s_]) for s_ in range(R)]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def med(fn):
        ts = []
        for it in range(iters + 3):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            torch.cuda.synchronize()
            if it >= 3:
                ts.append(e0.elapsed_time(e1) * 1e3)
        return sorted(ts)[len(ts) // 2]

    us_d = med(lambda: B.moe_ep_dispatch(peers, loc_d, k, d, status))
    us_c = med(lambda: B.moe_ep_combine(peers, loc_c, k, d, status))     # returns the received rows themselves: same bytes
    if status.cpu().tolist()[:2] != [0, 0]:
        raise SystemExit("ep emulation: device status")
    # the timed launches did the work: every arrival counter sits at its threshold, and combine, fed the received rows
    # themselves, returned k copies of every token to its rank (k * x exactly: a sum of k equal bf16 values in fp32)
    for s_ in range(R):
        want = torch.full_like(rcnt[s_], B.MOE_EP_BLOCK_ROWS)
        if rr[s_] % B.MOE_EP_BLOCK_ROWS:
            want[-1] = rr[s_] % B.MOE_EP_BLOCK_ROWS
        if not torch.equal(rcnt[s_], want) or not torch.equal(out[s_], (xs[s_].float() * k).to(torch.bfloat16)):
            raise SystemExit("ep emulation: wrong result")
    rows = sum(rr)
    by_d = 2.0 * cfg.T * d + 2.0 * rows * d + 16.0 * rows          # x once, every routed copy written once, its meta
    by_c = 2.0 * rows * d * 3 + 2.0 * cfg.T * d                      # y read, ret written and read back, out written
    return {"ranks": R, "tokens_per_rank": Tr, "rows": rows,
            "dispatch": {"us": us_d, "GBps": by_d / us_d / 1e3, "frac_of_hbm_peak": by_d / us_d / 1e3 / peaks["hbm_gbs"]},
            "combine": {"us": us_c, "GBps": by_c / us_c / 1e3, "frac_of_hbm_peak": by_c / us_c / 1e3 / peaks["hbm_gbs"]},
            "note": "ranks emulated on one GPU: local HBM stands in for peer memory; at 8 GPUs 7/8 of the rows would cross "
                    "NVLink (%.0f MB per GPU and direction)" % (2.0 * rows * d * 7 / 8 / R / 1e6)}


def respawn_under_launcher(n):
    """`python bench.py --gpus N` without a launcher: start the N ranks (one per GPU) and pass their output on."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


# ----------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=4, help="index of the headline workload (default: the training step)")
    ap.add_argument("--launch", default="fused", choices=["fused", "serial"],
                    help="launch mode of the headline value (default: the library's default, the persistent launch); "
                         "the other mode is timed too and reported beside it")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--fwd-only", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-compare", action="store_true", help="skip timing the other launch mode")
    ap.add_argument("--no-all-configs", action="store_true", help="skip the other workloads")
    ap.add_argument("--no-study", action="store_true", help="skip the SwiGLU+Add scheduling microbenchmark")
    ap.add_argument("--only-study", action="store_true", help="run the scheduling microbenchmark alone")
    ap.add_argument("--only-router", action="store_true", help="run the in-path router alone (on --config's shape)")
    ap.add_argument("--only-ep", action="store_true", help="run the emulated expert-parallel dispatch / combine alone")
    ap.add_argument("--study-iters", type=int, default=30)
    ap.add_argument("--plain-launch", action="store_true",
                    help="diagnostic: persistent launches without the cooperative launch attribute (for profiler captures)")
    ap.add_argument("--small", type=str, default="", help="T,d,F[,E]: reduced sizes of the chosen config (profiling captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    cfg = configs.CONFIGS[args.config]
    if args.small:
        v = [int(q) for q in args.small.split(",")]
        cfg = configs.small_variant(cfg, v[0], v[1], v[2], v[3] if len(v) > 3 else None)
    train = cfg.bwd and not args.fwd_only

    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) == 0:
            run_reference(args, cfg, train)
        return

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        respawn_under_launcher(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the layer has no CPU path)")

    if args.plain_launch:
        from paper_2605_23764_b200 import binding as B
        Workload.plain_launch = True
        B.moe_debug_set_plain_launch(None, True)
    if args.only_ep:
        torch.cuda.set_device(0)
        print(json.dumps({"ep_emulated": ep_emulated(cfg, load_peaks(), iters=args.study_iters)}), flush=True)
        return
    if args.only_router:
        torch.cuda.set_device(0)
        print(json.dumps({"router_in_path": router_in_path(cfg, load_peaks(), args.study_iters)}), flush=True)
        return
    if args.only_study:
        torch.cuda.set_device(0)
        print(json.dumps({"scheduling_study": scheduling_study(load_peaks(), args.study_iters)}), flush=True)
        return

    world, rank, local = dist_setup()
    if args.gpus != world and rank == 0:
        print(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s); reporting n_gpus={world}",
              file=sys.stderr)
    torch.cuda.set_device(local)
    peaks = load_peaks()
    other_mode = "serial" if args.launch == "fused" else "fused"
    modes = [args.launch] if args.no_compare else [args.launch, other_mode]

    # ---- headline workload: device-resident timing of the launch modes (max over ranks) ----------
    wl = Workload(cfg, train)
    layers = {m: wl.make_layer(m) for m in modes}
    results = {m: wl.measure(layers[m], args.steps, args.warmup, world, local) for m in modes}
    head = args.launch
    layer, res = layers[head], results[head]
    roofline, step_roofline = rooflines(cfg, train, res, peaks)
    other = None
    if other_mode in results:
        r2 = results[other_mode]
        roof2, step2 = rooflines(cfg, train, r2, peaks)
        other = {"launch": LAUNCH_NAMES[other_mode], "ms_per_step": r2["ms_per_step"], "value": r2["value"],
                 "phases_ms": r2["phases_ms"], "roofline": roof2, "step_roofline": step2, "clocks": r2["clocks"]}
        layers[other_mode].close()

    # ---- end to end through the host-buffer entry points (headline launch mode) -------------------
    # In a training step the forward result may leave for the host while the backward computes
    # (MOE_FLAG_DEFER_OUT_COPY: out_host is complete when the following moe_ffn_bwd_host is).
    e2e = None
    if not args.no_e2e:
        e2e_layer = wl.make_layer(head, defer_out_copy=train)
        e2e = run_e2e(wl, e2e_layer, args.steps, world)
        e2e["out_copy"] = ("deferred behind the backward call (MOE_FLAG_DEFER_OUT_COPY); complete before the step's end"
                           if train else "in front of the call's end")
        e2e_layer.close()

    # ---- CPU oracle baseline (rank 0, single-GPU run only) ----------------------------------------
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        n_exp, rows = calibrate_sample(cfg, train, oracle.threads())
        secs, fl, desc = oracle_sample(cfg, train, n_exp, rows, inputs=wl.inp)
        cpu_baseline = {"value": fl / secs / 1e12, "unit": "TFLOP/s", "cores": oracle.threads(), "kind": "oracle",
                        "sample": desc, "seconds": secs}
    layer.close()

    # ---- the other workloads, both launch modes (forward-only configurations) ---------------------
    all_configs = None
    if not args.no_all_configs and not args.small:
        del wl, layers, layer
        gc.collect(); torch.cuda.empty_cache()
        all_configs = [{"workload": cfg.name, "launch_fused_ms": results.get("fused", {}).get("ms_per_step"),
                        "launch_serial_ms": results.get("serial", {}).get("ms_per_step"),
                        "fused": {"step_roofline": rooflines(cfg, train, results["fused"], peaks)[1],
                                  "clocks": results["fused"]["clocks"]} if "fused" in results else None,
                        "serial": {"step_roofline": rooflines(cfg, train, results["serial"], peaks)[1],
                                   "clocks": results["serial"]["clocks"]} if "serial" in results else None}]
        for ci in (1, 2, 3):
            if ci == args.config:
                continue
            c2 = configs.CONFIGS[ci]
            w2 = Workload(c2, False)
            entry = {"workload": c2.name}
            for m in ("fused", "serial"):
                lay = w2.make_layer(m)
                # the other workloads are timed for as long as the headline one (their steps are 4-40 times shorter)
                r = w2.measure(lay, args.steps, args.warmup, world, local, min_timed_ms=results[head]["timed_ms"])
                lay.close()
                roof_m, step_m = rooflines(c2, False, r, peaks)
                entry[f"launch_{m}_ms"] = r["ms_per_step"]
                entry[m] = {"value": r["value"], "step_roofline": step_m, "roofline": roof_m, "clocks": r["clocks"],
                            "phases_ms": r["phases_ms"], "steps": r["steps"]}
            all_configs.append(entry)
            del w2
            gc.collect(); torch.cuda.empty_cache()

    study = None
    if rank == 0 and world == 1 and not args.no_study and not args.small:
        study = scheduling_study(peaks, args.study_iters)
    router = None
    if rank == 0 and world == 1 and not args.no_study:
        router = router_in_path(cfg, peaks, args.study_iters)
    ep = None
    if rank == 0 and world == 1 and not args.no_study and cfg.S == 0:
        ep = ep_emulated(cfg, peaks, iters=args.study_iters)

    if rank == 0:
        desc = workload_desc(cfg, train)
        desc["launch"] = LAUNCH_NAMES[head]
        desc["launch_choice"] = "the library's default mode" if head == "fused" else "requested"
        desc["launches_per_step"] = res["launches"] / max(1, args.steps)
        line = {
            "metric": METRIC, "value": res["value"], "unit": "TFLOP/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": res["ms_per_step"],
            "us_per_layer": res["ms_per_step"] * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": desc, "clocks": res["clocks"], "e2e": e2e, "gpu_launches": res["launches"],
            "roofline": roofline, "step_roofline": step_roofline, "phases_ms": res["phases_ms"],
            "other_launch_mode": other, "all_configs": all_configs, "cpu_baseline": cpu_baseline,
            "scheduling_study": study, "router_in_path": router, "ep_emulated": ep,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
