"""GPU parity of the forward layer against the oracle, stage by stage on small cases and on
the output for the benchmark configurations (sampled tokens at full size)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_23764_b200 import MoeLayer
from tests.gpu_util import assert_close_bf16, small_problem
from workloads import configs

pytestmark = pytest.mark.gpu


def _fwd_case(T, d, E, k, S, F, seed, renorm=True, serial=False, stages=True):
    x, W1, W2, logits, _ = small_problem(T, d, E, k, S, F, seed)
    layer = MoeLayer(T, d, E, k, S, F, renorm=renorm, save_for_bwd=True, serial=serial)
    ids, w = layer.route(logits)
    out = layer.ffn_fwd(x, ids, w, W1, W2)
    torch.cuda.synchronize()
    assert layer.status() == (0, 0)
    ref_out, H, A, Y = oracle.fwd(x, ids.cpu(), w.cpu(), W1, W2, S=S, save=True)
    if stages:
        kp = k + S
        prow = layer.debug("prow_of")[:T * kp].long()
        cap = layer.debug("Xp").numel() // d
        Xp = layer.debug("Xp").view(cap, d)[prow]
        tok = torch.arange(T * kp, device="cuda") // kp
        assert torch.equal(Xp, x[tok]), "gather"
        wfull = torch.cat([w, torch.ones(T, S, device="cuda")], 1).reshape(-1, 1).double().cpu().numpy()
        assert_close_bf16(layer.debug("H").view(cap, 2 * F)[prow], H, "H = x.W_gate_up")
        assert_close_bf16(layer.debug("A").view(cap, F)[prow], A * wfull, "A = w*silu(g)*u")
        assert_close_bf16(layer.debug("Y").view(cap, d)[prow], Y * wfull, "Y = A.W_down")
    assert_close_bf16(out, ref_out, "out")
    layer.close()
    return out


@pytest.mark.parametrize("serial", [False, True])
def test_config0(serial):
    c = configs.CONFIGS[0]
    inp = configs.make_inputs(c, "cuda")
    layer = MoeLayer(c.T, c.d, c.E, c.k, c.S, c.F, renorm=c.renorm, save_for_bwd=True, serial=serial)
    ids, w = layer.route(inp["logits"])
    out = layer.ffn_fwd(inp["x"], ids, w, inp["W_gate_up"], inp["W_down"])
    ref = oracle.fwd(inp["x"], ids.cpu(), w.cpu(), inp["W_gate_up"], inp["W_down"])
    assert layer.status() == (0, 0)
    assert_close_bf16(out, ref, "config 0 out")
    layer.close()


@pytest.mark.parametrize("T,d,E,k,S,F", [
    (256, 256, 8, 2, 0, 128),     # config 0 shape
    (300, 264, 10, 3, 1, 200),    # ragged everything: K tail, N tails, F not a tile multiple
    (1, 64, 4, 2, 0, 64),         # a single token
    (515, 128, 3, 1, 2, 320),     # experts spanning several M-blocks, shared experts
    (64, 512, 40, 4, 0, 72),      # more experts than rows per expert: many empty / tiny segments
])
@pytest.mark.parametrize("serial", [False, True])
def test_small_shapes_stagewise(T, d, E, k, S, F, serial):
    _fwd_case(T, d, E, k, S, F, seed=T + F, serial=serial)


def test_single_expert_is_dense_ffn():
    T, d, F = 384, 192, 256
    x, W1, W2, _, _ = small_problem(T, d, 1, 1, 0, F, 5)
    layer = MoeLayer(T, d, 1, 1, 0, F)
    ids = torch.zeros(T, 1, dtype=torch.int32, device="cuda")
    w = torch.ones(T, 1, dtype=torch.float32, device="cuda")
    out = layer.ffn_fwd(x, ids, w, W1, W2)
    xd, W1d, W2d = x.double(), W1[0].double(), W2[0].double()
    dense = (torch.nn.functional.silu(xd @ W1d[:F].T) * (xd @ W1d[F:].T)) @ W2d.T
    assert_close_bf16(out, dense.cpu().numpy(), "dense FFN")
    layer.close()


def test_zero_weights_and_empty_batch():
    T, d, E, k, F = 100, 64, 4, 2, 64
    x, W1, W2, logits, _ = small_problem(T, d, E, k, 0, F, 9)
    layer = MoeLayer(T, d, E, k, 0, F)
    ids, w = layer.route(logits)
    out = layer.ffn_fwd(x, ids, torch.zeros_like(w), W1, W2)
    assert torch.count_nonzero(out).item() == 0
    out0 = layer.ffn_fwd(x[:0], ids[:0], w[:0], W1, W2)
    assert out0.shape == (0, d)
    # a smaller batch than T_max on the same context
    out_small = layer.ffn_fwd(x[:37].contiguous(), ids[:37].contiguous(), w[:37].contiguous(), W1, W2)
    ref = oracle.fwd(x[:37], ids[:37].cpu(), w[:37].cpu(), W1, W2)
    assert_close_bf16(out_small, ref, "T < T_max")
    layer.close()


def _sampled_tokens_check(cfg, n_tokens=24, serial=False):
    """Full-size forward on the GPU; the oracle evaluates a sample of tokens one by one."""
    inp = configs.make_inputs(cfg, "cuda")
    layer = MoeLayer(cfg.T, cfg.d, cfg.E, cfg.k, cfg.S, cfg.F, renorm=cfg.renorm, serial=serial)
    ids, w = layer.route(inp["logits"])
    out = layer.ffn_fwd(inp["x"], ids, w, inp["W_gate_up"], inp["W_down"])
    torch.cuda.synchronize()
    assert layer.status() == (0, 0)
    assert torch.isfinite(out.float()).all()
    if not serial:  # the one-launch-per-operator mode must give the same bits (same tile math)
        other = MoeLayer(cfg.T, cfg.d, cfg.E, cfg.k, cfg.S, cfg.F, renorm=cfg.renorm, serial=True)
        out_serial = other.ffn_fwd(inp["x"], ids, w, inp["W_gate_up"], inp["W_down"])
        assert other.status() == (0, 0)
        assert torch.equal(out, out_serial), "fused and serial launches disagree"
        other.close()
    ids_c, w_c = ids.cpu(), w.cpu()
    counts = torch.bincount(ids_c.flatten().long(), minlength=cfg.E)
    order = torch.argsort(counts)
    nonempty = order[counts[order] > 0]
    picks = set()
    for e in (int(nonempty[0]), int(nonempty[-1])):  # a token of the least and of the most loaded expert
        picks.add(int(torch.nonzero((ids_c == e).any(1))[0]))
    g = torch.Generator().manual_seed(cfg.seed)
    picks |= set(torch.randint(0, cfg.T, (n_tokens,), generator=g).tolist())
    picks |= {0, cfg.T - 1}
    got, want = [], []
    for t in sorted(picks):
        es = ids_c[t].long().tolist() + list(range(cfg.E, cfg.Ep))
        W1 = inp["W_gate_up"][es].cpu()
        W2 = inp["W_down"][es].cpu()
        sub_ids = torch.arange(cfg.k, dtype=torch.int32)[None]
        ref = oracle.fwd(inp["x"][t:t + 1].cpu(), sub_ids, w_c[t:t + 1], W1, W2, S=cfg.S)
        want.append(ref[0])
        got.append(out[t].double().cpu().numpy())
    assert_close_bf16(np.stack(got), np.stack(want), f"{cfg.name} sampled tokens")
    layer.close()


@pytest.mark.parametrize("idx", [1, 2, 3, 4])
def test_benchmark_configs_full_size_sampled(idx):
    _sampled_tokens_check(configs.CONFIGS[idx])
