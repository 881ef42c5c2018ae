"""Helpers of the GPU parity tests: tolerances of the bf16 path and oracle-side sampling."""
import numpy as np
import torch

MAX_REL = 2e-2    # max|err| <= MAX_REL * max|ref|
MEAN_REL = 5e-3   # sum|err| / sum|ref| <= MEAN_REL


def err_stats(got, ref):
    got = got.detach().double().cpu().numpy() if hasattr(got, "detach") else np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    err = np.abs(got - ref)
    mx = float(err.max()) / max(float(np.abs(ref).max()), 1e-300) if err.size else 0.0
    mean = float(err.sum()) / max(float(np.abs(ref).sum()), 1e-300) if err.size else 0.0
    return mx, mean


def assert_close_bf16(got, ref, what, max_rel=MAX_REL, mean_rel=MEAN_REL):
    mx, mean = err_stats(got, ref)
    assert np.isfinite(mx) and np.isfinite(mean), f"{what}: non-finite values"
    assert mx <= max_rel and mean <= mean_rel, f"{what}: max-rel {mx:.3e} (<= {max_rel}), mean-rel {mean:.3e} (<= {mean_rel})"


def small_problem(T, d, E, k, S, F, seed, renorm=True, device="cuda"):
    """Random bf16 problem + fp32 logits on `device` (torch generator; used for odd shapes)."""
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(T, d, generator=g).to(torch.bfloat16)
    W1 = (torch.randn(E + S, 2 * F, d, generator=g) / d ** 0.5).to(torch.bfloat16)
    W2 = (torch.randn(E + S, d, F, generator=g) / d ** 0.5).to(torch.bfloat16)
    logits = torch.randn(T, E, generator=g)
    dout = torch.randn(T, d, generator=g).to(torch.bfloat16)
    return [t.to(device) for t in (x, W1, W2, logits, dout)]
