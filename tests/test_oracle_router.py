"""Pins of the oracle's in-path router (Section 2.2, router description): linear scores, softmax top-k on them, and the
gradient of the k scores w.r.t. the logits.  CPU only; nothing here comes from the CUDA path."""
import numpy as np
import pytest
import torch

import oracle


def test_logits_are_the_matrix_product_with_the_router_weights_transposed():
    g = torch.Generator().manual_seed(3)
    x = torch.randn(7, 5, generator=g, dtype=torch.float64)
    W = torch.randn(3, 5, generator=g, dtype=torch.float64)     # [E, d]: not square, so a transposed operand cannot pass
    got = oracle.router_logits(x, W)
    np.testing.assert_allclose(got, (x @ W.T).numpy(), rtol=1e-14, atol=1e-14)
    # hand-built: token 0 = unit vector c picks column c of W_r
    x1 = np.zeros((1, 5)); x1[0, 2] = 2.0
    np.testing.assert_array_equal(oracle.router_logits(x1, W), 2.0 * W.numpy()[None, :, 2])


def test_router_fwd_is_route_on_the_rounded_logits():
    g = torch.Generator().manual_seed(4)
    x = torch.randn(33, 16, generator=g).to(torch.bfloat16)
    W = (torch.randn(12, 16, generator=g) * 0.3).to(torch.bfloat16)
    ids, w, logits = oracle.router_fwd(x, W, 3, True)
    ref = torch.topk(torch.from_numpy(logits), 3, dim=1)
    assert np.array_equal(ids, ref.indices.numpy().astype(np.int32))          # no ties in this data
    p = torch.softmax(torch.from_numpy(logits), dim=1).gather(1, ref.indices)
    np.testing.assert_allclose(w, (p / p.sum(1, keepdim=True)).numpy(), rtol=1e-6)


def _autograd(logits, ids, g, renorm):
    l = torch.tensor(logits, dtype=torch.float64, requires_grad=True)
    p = torch.softmax(l, dim=1).gather(1, torch.from_numpy(ids.astype(np.int64)))
    if renorm:
        p = p / p.sum(1, keepdim=True)
    (p * torch.from_numpy(g)).sum().backward()
    return l.grad.numpy()


@pytest.mark.parametrize("renorm", [False, True])
@pytest.mark.parametrize("T,E,k", [(9, 8, 2), (5, 16, 6), (4, 5, 5), (6, 7, 1)])
def test_router_bwd_matches_autograd_of_softmax_gather(T, E, k, renorm):
    rng = np.random.default_rng(10 * T + E + k)
    logits = rng.normal(size=(T, E)).astype(np.float32)        # fp32 values: the oracle reads fp32 logits exactly
    ids, _ = oracle.route(logits, k, renorm)
    g = rng.normal(size=(T, k))
    got = oracle.router_bwd(logits, ids, g, renorm)
    np.testing.assert_allclose(got, _autograd(logits, ids, g, renorm), rtol=1e-11, atol=1e-13)
    # softmax is shift invariant: the gradient of every row sums to zero
    np.testing.assert_allclose(got.sum(1), 0.0, atol=1e-13)
    if renorm:
        mask = np.ones((T, E), bool)
        np.put_along_axis(mask, ids.astype(np.int64), False, axis=1)
        assert np.all(got[mask] == 0.0)                          # a softmax over the selected experts only
        if k == 1:
            assert np.all(got == 0.0)                            # a single renormalised score is the constant 1


def test_router_bwd_finite_differences_of_the_scores():
    rng = np.random.default_rng(5)
    T, E, k = 3, 6, 3
    logits = rng.normal(size=(T, E)).astype(np.float32) * 2
    ids, _ = oracle.route(logits, k, False)
    g = rng.normal(size=(T, k))

    def scores(l):                                               # closed form, selection held fixed
        e = np.exp(l - l.max(1, keepdims=True))
        return np.take_along_axis(e / e.sum(1, keepdims=True), ids.astype(np.int64), axis=1)

    got = oracle.router_bwd(logits, ids, g, False)
    l64 = logits.astype(np.float64)
    for t in range(T):
        for e in range(E):
            h = 1e-6
            lp, lm = l64.copy(), l64.copy()
            lp[t, e] += h; lm[t, e] -= h
            fd = ((scores(lp) - scores(lm)) * g).sum() / (2 * h)
            assert abs(fd - got[t, e]) <= 1e-8 * max(1.0, abs(fd))


# ---- sigmoid gating variant
@pytest.mark.parametrize("renorm", [False, True])
def test_sigmoid_route_matches_torch_sigmoid_topk(renorm):
    rng = np.random.default_rng(12)
    logits = (rng.normal(size=(40, 16)) * 2).astype(np.float32)
    ids, w = oracle.route(logits, 4, renorm, gate="sigmoid")
    l = torch.from_numpy(logits).double()
    ref = torch.topk(l, 4, dim=1)
    assert np.array_equal(ids, ref.indices.numpy().astype(np.int32))           # same selection as the softmax gate
    assert np.array_equal(ids, oracle.route(logits, 4, renorm)[0])
    s = torch.sigmoid(ref.values)
    if renorm:
        s = s / s.sum(1, keepdim=True)
    np.testing.assert_allclose(w, s.numpy(), rtol=1e-14)
    # closed forms: l = 0 -> 1/2, l = ln 3 -> 3/4; per-expert scores do not depend on the other logits
    one = np.array([[0.0, np.log(3.0), -50.0, -60.0]], dtype=np.float32)
    _, w1 = oracle.route(one, 2, False, gate="sigmoid")
    np.testing.assert_allclose(w1, [[0.75, 0.5]], rtol=1e-7)
    other = one.copy(); other[0, 2] = -1.0
    np.testing.assert_array_equal(oracle.route(other, 2, False, gate="sigmoid")[1], w1)


@pytest.mark.parametrize("renorm", [False, True])
@pytest.mark.parametrize("T,E,k", [(9, 8, 2), (5, 16, 6), (6, 7, 1)])
def test_sigmoid_router_bwd_matches_autograd(T, E, k, renorm):
    rng = np.random.default_rng(3 * T + E + k)
    logits = rng.normal(size=(T, E)).astype(np.float32)
    ids, _ = oracle.route(logits, k, renorm, gate="sigmoid")
    g = rng.normal(size=(T, k))
    got = oracle.router_bwd(logits, ids, g, renorm, gate="sigmoid")
    l = torch.tensor(logits, dtype=torch.float64, requires_grad=True)
    s = torch.sigmoid(l).gather(1, torch.from_numpy(ids.astype(np.int64)))
    if renorm:
        s = s / s.sum(1, keepdim=True)
    (s * torch.from_numpy(g)).sum().backward()
    np.testing.assert_allclose(got, l.grad.numpy(), rtol=1e-11, atol=1e-14)
    mask = np.ones((T, E), bool)
    np.put_along_axis(mask, ids.astype(np.int64), False, axis=1)
    assert np.all(got[mask] == 0.0)
    if renorm and k == 1:
        assert np.all(np.abs(got) < 1e-15)
