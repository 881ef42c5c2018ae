"""Router in the path (Section 2.2, router description): x W_r^T on the tensor cores with the softmax top-k in the
same launch, and the gradient of the scores w.r.t. the logits, against the fp64 oracle."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _inputs(T, d, E, seed, dup=None):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(T, d, generator=g).to(torch.bfloat16)
    W = (torch.randn(E, d, generator=g) * 0.02).to(torch.bfloat16)
    if dup:                                   # experts with identical weights: exactly equal logits, whatever the sum order
        for a, b in dup:
            W[b] = W[a]
    return x, W


def _run_fwd(T, d, E, k, renorm, x, W, want_logits=True):
    from paper_2605_23764_b200 import MoeLayer, binding as B
    dev = torch.device("cuda:0")
    layer = MoeLayer(T, d, E, k, 0, 128, renorm=renorm)
    ids = torch.full((T, k), -7, dtype=torch.int32, device=dev)
    w = torch.full((T, k), float("nan"), dtype=torch.float32, device=dev)
    logits = torch.full((T, E), float("nan"), dtype=torch.float32, device=dev) if want_logits else None
    counts = torch.full((E,), -1, dtype=torch.int32, device=dev)
    B.moe_router_fwd(layer.ctx, x.to(dev), W.to(dev), T, ids, w, logits, counts)
    torch.cuda.synchronize()
    assert layer.status() == (0, 0)
    return layer, ids.cpu().numpy(), w.cpu().numpy(), None if logits is None else logits.cpu().numpy(), counts.cpu().numpy()


@pytest.mark.parametrize("T,d,E,k,renorm", [
    (300, 256, 8, 2, True),          # one ragged tile, E below the smallest MMA width
    (1000, 2048, 64, 6, False),      # four tiles, the last one ragged
    (517, 520, 40, 3, True),         # d not a multiple of the 64-wide k-block, E not a multiple of 16
    (256, 64, 256, 8, True),         # one k-block, the widest accumulator
    (4096, 7168, 256, 8, True),      # the routing of config 2 / 4 at full width (T of config 2)
])
def test_router_fwd_against_the_oracle(T, d, E, k, renorm):
    import oracle
    x, W = _inputs(T, d, E, 7 * T + E)
    layer, ids, w, logits, counts = _run_fwd(T, d, E, k, renorm, x, W)
    ids_ref, w_ref, logits_ref = oracle.router_fwd(x, W, k, renorm)

    # 1. logits: fp32 accumulation of d exact products; |err| <= d * 2^-23 * sum |x_c W_ec| covers any summation order and
    #    truncating adds, and is orders of magnitude below what a dropped k-block or a wrong operand would give
    mag = np.abs(x.double().numpy()) @ np.abs(W.double().numpy()).T
    err = np.abs(logits.astype(np.float64) - logits_ref)
    assert np.all(err <= d * 2.0 ** -23 * mag + 1e-30), (err.max(), (d * 2.0 ** -23 * mag).min())
    assert np.sqrt((err ** 2).mean()) <= 2e-6 * np.sqrt((logits_ref ** 2).mean()) * max(1.0, np.sqrt(d / 256))

    # 2. the selection and the scores, in the precision the kernel decides in: the oracle's routing of the kernel's own
    #    fp32 logits must come out bit for bit
    ids_same, w_same = oracle.route(logits, k, renorm)
    assert np.array_equal(ids, ids_same)
    np.testing.assert_allclose(w, w_same, rtol=2e-6, atol=1e-30)
    assert np.array_equal(counts, np.bincount(ids.reshape(-1), minlength=E))

    # 3. against the exact computation: only tokens whose decision hangs on a gap smaller than the rounding may differ
    srt = -np.sort(-logits_ref, axis=1)[:, :min(k + 1, E)]
    gap = np.min(srt[:, :-1] - srt[:, 1:], axis=1)
    clear = gap > 4 * err.max()
    assert clear.mean() > 0.95          # near-ties among 9 of 256 logits are not rare, but they are few
    assert np.array_equal(ids[clear], ids_ref[clear])
    np.testing.assert_allclose(w[clear], w_ref[clear], rtol=1e-4)
    layer.close()


def test_equal_logits_go_to_the_lower_expert_id():
    import oracle
    T, d, E, k = 200, 128, 16, 4
    x, W = _inputs(T, d, E, 99, dup=[(1, 9), (9, 14), (3, 5)])     # experts 1 = 9 = 14 and 3 = 5
    layer, ids, w, logits, _ = _run_fwd(T, d, E, k, False, x, W)
    assert np.array_equal(logits[:, 1], logits[:, 9]) and np.array_equal(logits[:, 9], logits[:, 14])
    ids_ref, w_ref = oracle.route(logits, k, False)
    assert np.array_equal(ids, ids_ref)
    # wherever 9 was selected, 1 sits right before it
    for t in range(T):
        row = list(ids[t])
        if 9 in row:
            assert row.index(1) == row.index(9) - 1
    layer.close()


def test_logits_are_optional():
    T, d, E, k = 130, 192, 24, 2
    x, W = _inputs(T, d, E, 5)
    layer, ids, w, logits, counts = _run_fwd(T, d, E, k, True, x, W)
    layer2, ids2, w2, none, counts2 = _run_fwd(T, d, E, k, True, x, W, want_logits=False)
    assert none is None and np.array_equal(ids, ids2) and np.array_equal(w, w2) and np.array_equal(counts, counts2)
    layer.close(); layer2.close()


@pytest.mark.parametrize("renorm", [False, True])
@pytest.mark.parametrize("T,E,k", [(333, 40, 3), (1000, 256, 8), (64, 8, 8), (50, 5, 1)])
def test_router_bwd_against_the_oracle(T, E, k, renorm):
    import oracle
    from paper_2605_23764_b200 import MoeLayer, binding as B
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(T + E + k)
    logits = (rng.normal(size=(T, E)) * 1.5).astype(np.float32)
    ids, _ = oracle.route(logits, k, renorm)
    g = rng.normal(size=(T, k)).astype(np.float32)
    ref = oracle.router_bwd(logits, ids, g, renorm)
    layer = MoeLayer(T, 64, E, k, 0, 128, renorm=renorm)
    out = torch.full((T, E), float("nan"), dtype=torch.float32, device=dev)
    B.moe_router_bwd(layer.ctx, torch.from_numpy(logits).to(dev), torch.from_numpy(ids).to(dev), torch.from_numpy(g).to(dev), T, out)
    torch.cuda.synchronize()
    got = out.cpu().numpy().astype(np.float64)
    # fp32 exp / divide / a k-term dot product: a few ulp of the largest term of each row
    scale = np.abs(ref).max(axis=1, keepdims=True) + np.abs(g).max(axis=1, keepdims=True) * 1e-3
    assert np.all(np.abs(got - ref) <= 2e-5 * scale + 1e-12)
    if renorm:
        mask = np.ones((T, E), bool)
        np.put_along_axis(mask, ids.astype(np.int64), False, axis=1)
        assert np.all(got[mask] == 0.0)
    layer.close()


def test_router_refuses_what_it_cannot_do():
    from paper_2605_23764_b200 import MoeLayer, binding as B
    dev = torch.device("cuda:0")
    layer = MoeLayer(64, 64, 300, 2, 0, 128)         # E > 256
    x = torch.zeros(64, 64, dtype=torch.bfloat16, device=dev)
    W = torch.zeros(300, 64, dtype=torch.bfloat16, device=dev)
    ids = torch.zeros(64, 2, dtype=torch.int32, device=dev)
    w = torch.zeros(64, 2, dtype=torch.float32, device=dev)
    with pytest.raises(B.MoeError):
        B.moe_router_fwd(layer.ctx, x, W, 64, ids, w)
    layer.close()


# ---- sigmoid gating variant (MOE_FLAG_SIGMOID_GATE): per-expert scores, the same selection
@pytest.mark.parametrize("renorm", [False, True])
def test_sigmoid_gate_in_route_router_fwd_and_bwd(renorm):
    import oracle
    from paper_2605_23764_b200 import MoeLayer, binding as B
    dev = torch.device("cuda:0")
    T, d, E, k = 700, 512, 48, 4
    x, W = _inputs(T, d, E, 31)
    layer = MoeLayer(T, d, E, k, 0, 128, renorm=renorm, sigmoid_gate=True)
    # moe_route on given logits
    g = torch.Generator().manual_seed(8)
    logits = (torch.randn(T, E, generator=g) * 2).contiguous()
    ids, w = layer.route(logits.to(dev))
    ids_ref, w_ref = oracle.route(logits.numpy(), k, renorm, gate="sigmoid")
    assert np.array_equal(ids.cpu().numpy(), ids_ref)
    np.testing.assert_allclose(w.cpu().numpy(), w_ref, rtol=2e-6)
    # router in the path
    ids2 = torch.empty(T, k, dtype=torch.int32, device=dev); w2 = torch.empty(T, k, dtype=torch.float32, device=dev)
    lg = torch.empty(T, E, dtype=torch.float32, device=dev)
    B.moe_router_fwd(layer.ctx, x.to(dev), W.to(dev), T, ids2, w2, lg)
    torch.cuda.synchronize()
    ids_same, w_same = oracle.route(lg.cpu().numpy(), k, renorm, gate="sigmoid")
    assert np.array_equal(ids2.cpu().numpy(), ids_same)
    np.testing.assert_allclose(w2.cpu().numpy(), w_same, rtol=2e-6)
    # score gradient
    gw = torch.randn(T, k, generator=g)
    out = torch.full((T, E), float("nan"), dtype=torch.float32, device=dev)
    B.moe_router_bwd(layer.ctx, lg, ids2, gw.to(dev), T, out)
    torch.cuda.synchronize()
    ref = oracle.router_bwd(lg.cpu().numpy(), ids_same, gw.numpy(), renorm, gate="sigmoid")
    got = out.cpu().numpy().astype(np.float64)
    scale = np.abs(ref).max(axis=1, keepdims=True) + np.abs(gw.numpy()).max(axis=1, keepdims=True) * 1e-3
    assert np.all(np.abs(got - ref) <= 2e-5 * scale + 1e-12)
    mask = np.ones((T, E), bool)
    np.put_along_axis(mask, ids_same.astype(np.int64), False, axis=1)
    assert np.all(got[mask] == 0.0)
    assert layer.status() == (0, 0)
    layer.close()
