"""Pins for the oracle's forward and backward: the single-expert case against the dense
SwiGLU FFN written with library routines, the general case against an expert-major torch
statement and its autograd gradients, central finite differences, structural invariants."""
import numpy as np
import pytest
import torch
import torch.nn.functional as Fn

import oracle
from tests.torch_ref import moe_ffn_torch
from workloads import configs


def _problem(T=24, d=16, E=6, k=3, S=0, F=8, seed=0, renorm=True):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(T, d, generator=g, dtype=torch.float64)
    Wgu = torch.randn(E + S, 2 * F, d, generator=g, dtype=torch.float64) / d ** 0.5
    Wd = torch.randn(E + S, d, F, generator=g, dtype=torch.float64) / d ** 0.5
    logits = torch.randn(T, E, generator=g, dtype=torch.float32)
    ids, w = oracle.route(logits, k, renorm)
    dout = torch.randn(T, d, generator=g, dtype=torch.float64)
    return x, torch.from_numpy(ids), torch.from_numpy(w), Wgu, Wd, dout


def test_single_expert_weight_one_is_dense_swiglu_ffn():
    T, d, F = 19, 12, 10
    g = torch.Generator().manual_seed(1)
    x = torch.randn(T, d, generator=g, dtype=torch.float64)
    Wg = torch.randn(F, d, generator=g, dtype=torch.float64)
    Wu = torch.randn(F, d, generator=g, dtype=torch.float64)
    Wd = torch.randn(d, F, generator=g, dtype=torch.float64)
    dense = (Fn.silu(x @ Wg.T) * (x @ Wu.T)) @ Wd.T
    ids = np.zeros((T, 1), np.int32)
    w = np.ones((T, 1))
    out = oracle.fwd(x, ids, w, torch.cat([Wg, Wu])[None], Wd[None])
    assert np.allclose(out, dense.numpy(), rtol=1e-12, atol=1e-12)
    # the same through a shared expert only (k = 1 routed expert with zero weights + 1 shared)
    Wgu2 = torch.stack([torch.randn(2 * F, d, generator=g, dtype=torch.float64), torch.cat([Wg, Wu])])
    Wd2 = torch.stack([torch.randn(d, F, generator=g, dtype=torch.float64), Wd])
    out2 = oracle.fwd(x, ids, np.zeros((T, 1)), Wgu2, Wd2, S=1)
    assert np.allclose(out2, dense.numpy(), rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("S,renorm", [(0, True), (2, False), (1, True)])
def test_forward_matches_expert_major_library_statement(S, renorm):
    x, ids, w, Wgu, Wd, _ = _problem(S=S, renorm=renorm, seed=3 + S)
    out, H, A, Y = oracle.fwd(x, ids, w, Wgu, Wd, S=S, save=True)
    ref = moe_ffn_torch(x, ids.long(), w, Wgu, Wd, S=S)
    assert np.allclose(out, ref.numpy(), rtol=1e-11, atol=1e-12)
    # saved intermediates are consistent with each other
    F = Wgu.shape[1] // 2
    assert np.allclose(A, (Fn.silu(torch.from_numpy(H[:, :F])) * torch.from_numpy(H[:, F:])).numpy(), rtol=1e-12)
    kp = ids.shape[1] + S
    wfull = np.concatenate([w.numpy(), np.ones((x.shape[0], S))], axis=1).reshape(-1, 1)
    assert np.allclose((Y * wfull).reshape(x.shape[0], kp, -1).sum(1), out, rtol=1e-11, atol=1e-12)


def test_forward_structure():
    x, ids, w, Wgu, Wd, _ = _problem(seed=5)
    out = oracle.fwd(x, ids, w, Wgu, Wd)
    # linear in the routing weights
    w2 = torch.rand_like(w)
    lhs = oracle.fwd(x, ids, 2.0 * w + 3.0 * w2, Wgu, Wd)
    rhs = 2.0 * out + 3.0 * oracle.fwd(x, ids, w2, Wgu, Wd)
    assert np.allclose(lhs, rhs, rtol=1e-11, atol=1e-12)
    # permuting tokens permutes the output
    perm = torch.randperm(x.shape[0], generator=torch.Generator().manual_seed(2))
    assert np.allclose(oracle.fwd(x[perm], ids[perm], w[perm], Wgu, Wd), out[perm.numpy()], rtol=1e-13, atol=0)
    # relabelling experts (ids and weight slabs together) changes nothing
    E = Wgu.shape[0]
    relabel = torch.randperm(E, generator=torch.Generator().manual_seed(4))  # new id -> old id
    inv = torch.empty_like(relabel)
    inv[relabel] = torch.arange(E)
    out_r = oracle.fwd(x, inv[ids.long()].int(), w, Wgu[relabel], Wd[relabel])
    assert np.allclose(out_r, out, rtol=1e-13, atol=0)
    # zero down projection gives zero output; slot order inside a token does not matter beyond rounding
    assert np.all(oracle.fwd(x, ids, w, Wgu, torch.zeros_like(Wd)) == 0)
    assert np.allclose(oracle.fwd(x, ids.flip(1), w.flip(1), Wgu, Wd), out, rtol=1e-12, atol=1e-13)


def test_per_token_brute_force_tiny():
    x, ids, w, Wgu, Wd, _ = _problem(T=5, d=4, E=3, k=2, F=3, seed=9)
    out = oracle.fwd(x, ids, w, Wgu, Wd)
    F = 3
    for t in range(5):
        acc = [0.0] * 4
        for j in range(2):
            e = int(ids[t, j])
            h = [sum(float(x[t, c]) * float(Wgu[e, n, c]) for c in range(4)) for n in range(2 * F)]
            a = [h[f] / (1.0 + np.exp(-h[f])) * h[F + f] for f in range(F)]
            for c in range(4):
                acc[c] += float(w[t, j]) * sum(a[f] * float(Wd[e, c, f]) for f in range(F))
        assert np.allclose(out[t], acc, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("S", [0, 1])
def test_backward_matches_autograd(S):
    x, ids, w, Wgu, Wd, dout = _problem(S=S, seed=21 + S)
    xa, wa, W1, W2 = (t.clone().requires_grad_(True) for t in (x, w, Wgu, Wd))
    out = moe_ffn_torch(xa, ids.long(), wa, W1, W2, S=S)
    (out * dout).sum().backward()
    dx, dWgu, dWd, dw = oracle.bwd(dout, x, ids, w, Wgu, Wd, S=S)
    for got, want in ((dx, xa.grad), (dWgu, W1.grad), (dWd, W2.grad), (dw, wa.grad)):
        assert np.allclose(got, want.numpy(), rtol=1e-10, atol=1e-11)


def test_backward_central_finite_differences_config0():
    cfg = configs.CONFIGS[0]
    inp = configs.make_inputs(cfg)
    x, Wgu, Wd, dout = (inp[n].double() for n in ("x", "W_gate_up", "W_down", "dout"))
    ids, w = oracle.route(inp["logits"], cfg.k, cfg.renorm)
    w = torch.from_numpy(w)
    dx, dWgu, dWd, dw = oracle.bwd(dout, x, ids, w, Wgu, Wd)
    G = dout.numpy()

    def loss(x_, w_, W1_, W2_):
        return float((oracle.fwd(x_, ids, w_, W1_, W2_) * G).sum())

    rng = np.random.default_rng(0)
    h = 1e-4
    tensors = {"x": (x, dx), "w": (w, dw), "W1": (Wgu, dWgu), "W2": (Wd, dWd)}
    for name, (ten, grad) in tensors.items():
        flat_idx = rng.choice(ten.numel(), size=64 if name != "w" else 32, replace=False)
        for fi in flat_idx:
            args = {n: t for n, (t, _) in tensors.items()}
            plus, minus = ten.clone(), ten.clone()
            plus.view(-1)[fi] += h
            minus.view(-1)[fi] -= h
            args[name] = plus
            lp = loss(args["x"], args["w"], args["W1"], args["W2"])
            args[name] = minus
            lm = loss(args["x"], args["w"], args["W1"], args["W2"])
            fd = (lp - lm) / (2 * h)
            an = float(np.asarray(grad).reshape(-1)[fi])
            assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)), (name, int(fi), fd, an)


def test_backward_structure():
    x, ids, w, Wgu, Wd, dout = _problem(T=12, E=8, k=2, seed=33)
    ids = ids.clone()
    ids[ids == 5] = 6  # may duplicate an expert inside a token: still a valid input
    ids[ids == 2] = 3
    dx, dWgu, dWd, dw = oracle.bwd(dout, x, ids, w, Wgu, Wd)
    assert np.all(dWgu[5] == 0) and np.all(dWd[5] == 0) and np.all(dWgu[2] == 0) and np.all(dWd[2] == 0)
    # dx of a token depends only on that token's own upstream gradient
    dout2 = dout.clone()
    dout2[7] += 1.0
    dx2, *_ = oracle.bwd(dout2, x, ids, w, Wgu, Wd)
    keep = [t for t in range(12) if t != 7]
    assert np.array_equal(dx[keep], dx2[keep]) and not np.array_equal(dx[7], dx2[7])
    # adjoint identity <dout, J v> = <J^T dout, v> with J v by central differences on x
    v = torch.randn(x.shape, generator=torch.Generator().manual_seed(8), dtype=torch.float64)
    h = 1e-5
    jv = (oracle.fwd(x + h * v, ids, w, Wgu, Wd) - oracle.fwd(x - h * v, ids, w, Wgu, Wd)) / (2 * h)
    assert abs((dout.numpy() * jv).sum() - (dx * v.numpy()).sum()) < 1e-6 * abs((dx * v.numpy()).sum()) + 1e-8
