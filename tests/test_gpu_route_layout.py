"""GPU parity of routing and dispatch layout against the oracle: ids, counts, offsets and
permutation indices bit-exact; routing weights to fp32 rounding."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_23764_b200 import MoeLayer
from workloads import configs

pytestmark = pytest.mark.gpu


def _check_route_layout(logits, E, k, S, renorm):
    T = logits.shape[0]
    layer = MoeLayer(T, 64, E, k, S, 64, renorm=renorm)
    ids, w, counts = layer.route(logits, with_counts=True)
    ref_ids, ref_w = oracle.route(logits.cpu(), k, renorm)
    assert np.array_equal(ids.cpu().numpy(), ref_ids)
    assert np.allclose(w.cpu().numpy(), ref_w, rtol=2e-6, atol=1e-30)
    c, o, row_of, src_of = layer.layout(ids)
    rc, ro, rrow, rsrc = oracle.layout(ref_ids, E, S)
    assert np.array_equal(counts.cpu().numpy(), rc[:E])
    assert np.array_equal(c.cpu().numpy(), rc) and np.array_equal(o.cpu().numpy(), ro)
    assert np.array_equal(row_of.cpu().numpy(), rrow) and np.array_equal(src_of.cpu().numpy(), rsrc)
    assert layer.status() == (0, 0)
    layer.close()


@pytest.mark.parametrize("T,E,k,S,renorm", [(256, 8, 2, 0, True), (1000, 64, 6, 2, False), (4099, 256, 8, 1, True),
                                            (1, 4, 4, 0, True), (37, 5, 1, 0, False), (3000, 1000, 8, 0, True),
                                            (5, 40, 3, 3, True)])
def test_route_layout_random(T, E, k, S, renorm):
    g = torch.Generator().manual_seed(T + E)
    _check_route_layout(torch.randn(T, E, generator=g).cuda(), E, k, S, renorm)


def test_route_ties_and_extremes():
    l = torch.zeros(64, 16)
    l[1, 3] = l[1, 9] = 2.0
    l[2] = torch.arange(16).float()
    l[3, :] = -1e4
    l[3, 5] = 0.0
    l[4] = torch.round(torch.randn(16, generator=torch.Generator().manual_seed(1)) * 2) / 2  # many exact ties
    _check_route_layout(l.cuda(), 16, 4, 0, True)
    _check_route_layout(l.cuda(), 16, 16, 0, False)


def test_all_tokens_to_one_expert_and_empty_experts():
    T, E = 700, 12
    l = torch.full((T, E), -5.0)
    l[:, 7] = 5.0
    l[:, 2] = 1.0
    _check_route_layout(l.cuda(), E, 2, 0, True)


@pytest.mark.parametrize("idx", [0, 1, 2, 3, 4])
def test_benchmark_configs_full_size(idx):
    cfg = configs.CONFIGS[idx]
    x = configs.make_x(cfg, "cuda")
    logits = configs.make_logits(cfg, x)
    _check_route_layout(logits, cfg.E, cfg.k, cfg.S, cfg.renorm)
    if cfg.n_dead:
        ids, _ = oracle.route(logits.cpu(), cfg.k, cfg.renorm)
        counts, *_ = oracle.layout(ids, cfg.E, cfg.S)
        assert (counts == 0).sum() >= cfg.n_dead


def test_invalid_expert_id_is_reported_and_dropped():
    T, E, k = 100, 8, 2
    layer = MoeLayer(T, 64, E, k, 0, 64)
    ids = torch.randint(0, E, (T, k), dtype=torch.int32)
    ids[17, 1] = 99
    ids[50, 0] = -3
    c, o, row_of, src_of = layer.layout(ids.cuda())
    code, detail = layer.status()
    assert code == 1 and detail in (17 * k + 1, 50 * k)
    row_of = row_of.cpu().numpy()
    assert row_of[17 * k + 1] == -1 and row_of[50 * k] == -1
    assert c.sum().item() == T * k - 2 and o[-1].item() == T * k - 2
    assert layer.status() == (0, 0)  # reading clears the record
    layer.close()
