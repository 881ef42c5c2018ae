"""Pins for the oracle's routing and dispatch-layout functions: brute force, library
routines (torch.topk / softmax / stable argsort), closed-form special cases, invariants."""
import numpy as np
import pytest
import torch

import oracle
from workloads import configs


def _logits(T, E, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(T, E, generator=g, dtype=torch.float32)


@pytest.mark.parametrize("T,E,k", [(64, 8, 2), (33, 64, 6), (17, 256, 8), (5, 7, 7), (9, 5, 1)])
def test_topk_ids_brute_force(T, E, k):
    l = _logits(T, E, T * 1000 + E)
    ids, _ = oracle.route(l, k, renorm=False)
    for t in range(T):
        row = l[t].tolist()
        want = sorted(range(E), key=lambda e: (-row[e], e))[:k]
        assert ids[t].tolist() == want


def test_topk_ties_go_to_lower_id_and_slots_descend():
    l = torch.tensor([[1.0, 3.0, 3.0, 0.5, 3.0, 1.0],
                      [0.0, 0.0, 0.0, 0.0, 0.0, 0.0],
                      [-1.0, 2.0, -1.0, 2.0, 5.0, 5.0]], dtype=torch.float32)
    ids, w = oracle.route(l, 4, renorm=False)
    assert ids.tolist() == [[1, 2, 4, 0], [0, 1, 2, 3], [4, 5, 1, 3]]
    assert np.all(np.diff(w, axis=1) <= 0)


def test_k1_is_argmax_and_kE_is_full_sort():
    l = _logits(50, 16, 3)
    ids1, w1 = oracle.route(l, 1, renorm=True)
    assert ids1[:, 0].tolist() == torch.argmax(l, dim=1).tolist()
    assert np.allclose(w1, 1.0)
    idsE, wE = oracle.route(l, 16, renorm=False)
    assert idsE.tolist() == torch.argsort(l, dim=1, descending=True, stable=True).tolist()
    assert np.allclose(wE.sum(1), 1.0, atol=1e-12)  # full softmax sums to one


@pytest.mark.parametrize("renorm", [False, True])
def test_weights_match_library_softmax_topk(renorm):
    l = _logits(128, 64, 11)
    ids, w = oracle.route(l, 6, renorm)
    p = torch.softmax(l.double(), dim=1)
    vals, idx = torch.topk(p, 6, dim=1)
    if renorm:
        vals = vals / vals.sum(1, keepdim=True)
    assert ids.tolist() == idx.tolist()  # random logits: no ties
    assert np.allclose(w, vals.numpy(), rtol=1e-12, atol=0)
    if renorm:
        assert np.allclose(w.sum(1), 1.0, atol=1e-12)


def test_softmax_is_shift_invariant_and_safe_for_large_logits():
    l = _logits(8, 16, 5)
    _, w0 = oracle.route(l, 4, False)
    _, w1 = oracle.route(l + 1000.0, 4, False)  # exact shift in fp32 would change values; use small ints
    li = torch.round(l * 4) / 4
    _, a = oracle.route(li, 4, False)
    _, b = oracle.route(li + 64.0, 4, False)
    assert np.allclose(a, b, rtol=1e-12)
    assert np.all(np.isfinite(w1)) and np.all(np.isfinite(w0))


@pytest.mark.parametrize("T,E,k,S", [(64, 8, 2, 0), (100, 16, 4, 2), (7, 40, 3, 1), (1, 4, 4, 0)])
def test_layout_invariants_and_stable_sort(T, E, k, S):
    ids, _ = oracle.route(_logits(T, E, 17 + T), k, False)
    counts, offsets, row_of, src_of = oracle.layout(ids, E, S)
    kp = k + S
    n = T * kp
    assert counts.sum() == n and offsets[0] == 0 and offsets[-1] == n
    assert np.array_equal(np.diff(offsets), counts)
    assert np.all(counts[E:] == T)
    assert sorted(row_of.tolist()) == list(range(n))  # bijection
    assert np.array_equal(src_of[row_of], np.arange(n))
    # library pin: stable argsort of the per-slot expert id
    flat = np.concatenate([ids, np.tile(np.arange(E, E + S, dtype=np.int32), (T, 1))], axis=1).reshape(-1)
    assert np.array_equal(np.bincount(flat, minlength=E + S), counts)
    order = np.argsort(flat, kind="stable")
    assert np.array_equal(src_of, order)
    # gather then scatter of an iota tensor is the identity
    iota = np.arange(n)
    assert np.array_equal(iota[src_of][row_of], iota)
    for e in range(E + S):  # rows of a segment keep slot order
        seg = src_of[offsets[e]:offsets[e + 1]]
        assert np.all(np.diff(seg) > 0)


def test_layout_degenerate_cases():
    ids = np.full((10, 1), 3, np.int32)  # every token to one expert
    counts, offsets, row_of, src_of = oracle.layout(ids, 5, 0)
    assert counts.tolist() == [0, 0, 0, 10, 0]
    assert row_of.tolist() == list(range(10)) and src_of.tolist() == list(range(10))
    with pytest.raises(ValueError):
        oracle.layout(np.array([[7]], np.int32), 5, 0)
    with pytest.raises(ValueError):
        oracle.layout(np.array([[-1]], np.int32), 5, 0)


def test_config_routing_recipes():
    """Balanced configs give every expert tokens; the skewed one leaves the dead experts empty."""
    cfg = configs.small_variant(configs.CONFIGS[2], T=1024, d=256, F=64, E=32)
    x = configs.make_x(cfg)
    ids, w = oracle.route(configs.make_logits(cfg, x), cfg.k, cfg.renorm)
    counts, *_ = oracle.layout(ids, cfg.E, cfg.S)
    assert counts.sum() == cfg.T * cfg.kp and counts[:cfg.E].min() > 0 and counts[cfg.E] == cfg.T
    cfg3 = configs.small_variant(configs.CONFIGS[3], T=1024, d=4096, F=64)
    x = configs.make_x(cfg3)
    ids, _ = oracle.route(configs.make_logits(cfg3, x), cfg3.k, cfg3.renorm)
    counts, *_ = oracle.layout(ids, cfg3.E, cfg3.S)
    assert (counts == 0).sum() >= cfg3.n_dead
