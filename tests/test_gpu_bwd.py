"""GPU parity of the backward layer against the oracle: small cases element by element,
config 0 in full, the training-step configuration on sampled tokens and sampled experts."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_23764_b200 import MoeLayer
from tests.gpu_util import assert_close_bf16, small_problem
from workloads import configs

pytestmark = pytest.mark.gpu


def _bwd_case(T, d, E, k, S, F, seed, renorm=True, serial=False):
    x, W1, W2, logits, dout = small_problem(T, d, E, k, S, F, seed)
    layer = MoeLayer(T, d, E, k, S, F, renorm=renorm, save_for_bwd=True, serial=serial)
    ids, w = layer.route(logits)
    layer.ffn_fwd(x, ids, w, W1, W2)
    dx, dW1, dW2, dw = layer.ffn_bwd(dout, x, ids, w, W1, W2)
    torch.cuda.synchronize()
    assert layer.status() == (0, 0)
    rdx, rdW1, rdW2, rdw = oracle.bwd(dout, x, ids.cpu(), w.cpu(), W1, W2, S=S)
    assert_close_bf16(dx, rdx, "dx")
    assert_close_bf16(dW1, rdW1, "dW_gate_up")
    assert_close_bf16(dW2, rdW2, "dW_down")
    assert_close_bf16(dw, rdw, "d_topk_w")
    counts = np.bincount(ids.cpu().numpy().reshape(-1), minlength=E)
    for e in np.nonzero(counts == 0)[0]:  # experts without tokens get exact zeros
        assert torch.count_nonzero(dW1[e]).item() == 0 and torch.count_nonzero(dW2[e]).item() == 0
    layer.close()


@pytest.mark.parametrize("T,d,E,k,S,F", [
    (256, 256, 8, 2, 0, 128),
    (300, 264, 10, 3, 1, 200),
    (1, 64, 4, 2, 0, 64),
    (515, 128, 3, 1, 2, 320),
    (64, 512, 40, 4, 0, 72),
])
@pytest.mark.parametrize("serial", [False, True])
def test_small_shapes(T, d, E, k, S, F, serial):
    _bwd_case(T, d, E, k, S, F, seed=T + F, serial=serial)


@pytest.mark.parametrize("serial", [False, True])
def test_config0_full(serial):
    c = configs.CONFIGS[0]
    inp = configs.make_inputs(c, "cuda")
    layer = MoeLayer(c.T, c.d, c.E, c.k, c.S, c.F, renorm=c.renorm, save_for_bwd=True, serial=serial)
    ids, w = layer.route(inp["logits"])
    layer.ffn_fwd(inp["x"], ids, w, inp["W_gate_up"], inp["W_down"])
    dx, dW1, dW2, dw = layer.ffn_bwd(inp["dout"], inp["x"], ids, w, inp["W_gate_up"], inp["W_down"])
    rdx, rdW1, rdW2, rdw = oracle.bwd(inp["dout"], inp["x"], ids.cpu(), w.cpu(), inp["W_gate_up"], inp["W_down"])
    assert layer.status() == (0, 0)
    for got, ref, name in ((dx, rdx, "dx"), (dW1, rdW1, "dW_gate_up"), (dW2, rdW2, "dW_down"), (dw, rdw, "d_topk_w")):
        assert_close_bf16(got, ref, "config 0 " + name)
    layer.close()


def test_backward_needs_a_saved_forward():
    from paper_2605_23764_b200 import MoeError
    T, d, E, k, F = 64, 64, 4, 2, 64
    x, W1, W2, logits, dout = small_problem(T, d, E, k, 0, F, 3)
    layer = MoeLayer(T, d, E, k, 0, F, save_for_bwd=True)
    ids, w = layer.route(logits)
    with pytest.raises(MoeError):
        layer.ffn_bwd(dout, x, ids, w, W1, W2)
    layer.close()
    layer = MoeLayer(T, d, E, k, 0, F, save_for_bwd=False)
    layer.ffn_fwd(x, ids, w, W1, W2)
    with pytest.raises(MoeError):
        layer.ffn_bwd(dout, x, ids, w, W1, W2)
    layer.close()


def test_repeat_runs_and_launch_modes_are_bit_identical():
    """Five runs of the persistent launch and two of the operator-by-operator launches give the same
    bits: the tile math is shared and every reduction has a fixed order (a cheap race detector)."""
    T, d, E, k, S, F = 700, 256, 16, 4, 1, 256
    x, W1, W2, logits, dout = small_problem(T, d, E, k, S, F, 77)
    first = None
    for serial, reps in ((False, 5), (True, 2)):
        layer = MoeLayer(T, d, E, k, S, F, save_for_bwd=True, serial=serial)
        ids, w = layer.route(logits)
        for _ in range(reps):
            out = layer.ffn_fwd(x, ids, w, W1, W2)
            res = (out,) + layer.ffn_bwd(dout, x, ids, w, W1, W2)
            res = [r.clone() for r in res]
            assert layer.status() == (0, 0)
            if first is None:
                first = res
            else:
                for a, b in zip(first, res):
                    assert torch.equal(a, b)
        assert layer.launches() == (7 if serial else 1)   # launches of the backward call
        layer.close()


def test_training_config_full_size_sampled():
    cfg = configs.CONFIGS[4]
    inp = configs.make_inputs(cfg, "cuda")
    x, W1, W2, dout = inp["x"], inp["W_gate_up"], inp["W_down"], inp["dout"]
    layer = MoeLayer(cfg.T, cfg.d, cfg.E, cfg.k, cfg.S, cfg.F, renorm=cfg.renorm, save_for_bwd=True)
    ids, w = layer.route(inp["logits"])
    out = layer.ffn_fwd(x, ids, w, W1, W2)
    dx, dW1, dW2, dw = layer.ffn_bwd(dout, x, ids, w, W1, W2)
    torch.cuda.synchronize()
    assert layer.status() == (0, 0)
    ids_c, w_c = ids.cpu(), w.cpu()

    def check_against_oracle(out, dx, dW1, dW2, dw, what):
        # sampled tokens: out, dx and d_topk_w need only the token's own k experts
        g = torch.Generator().manual_seed(cfg.seed)
        toks = sorted(set(torch.randint(0, cfg.T, (10,), generator=g).tolist()) | {0, cfg.T - 1})
        got_o, want_o, got_dx, want_dx, got_dw, want_dw = [], [], [], [], [], []
        sub_ids = torch.arange(cfg.k, dtype=torch.int32)[None]
        for t in toks:
            es = ids_c[t].long().tolist()
            W1s, W2s = W1[es].cpu(), W2[es].cpu()
            want_o.append(oracle.fwd(x[t:t + 1].cpu(), sub_ids, w_c[t:t + 1], W1s, W2s)[0])
            rdx, _, _, rdw = oracle.bwd(dout[t:t + 1].cpu(), x[t:t + 1].cpu(), sub_ids, w_c[t:t + 1], W1s, W2s)
            want_dx.append(rdx[0]); want_dw.append(rdw[0])
            got_o.append(out[t].double().cpu().numpy()); got_dx.append(dx[t].double().cpu().numpy())
            got_dw.append(dw[t].double().cpu().numpy())
        assert_close_bf16(np.stack(got_o), np.stack(want_o), f"cfg4 {what} out (sampled tokens)")
        assert_close_bf16(np.stack(got_dx), np.stack(want_dx), f"cfg4 {what} dx (sampled tokens)")
        assert_close_bf16(np.stack(got_dw), np.stack(want_dw), f"cfg4 {what} d_topk_w (sampled tokens)")
        # sampled experts: a weight gradient needs only the rows of its expert
        counts = torch.bincount(ids_c.flatten().long(), minlength=cfg.E)
        order = torch.argsort(counts)
        for e in (int(order[0]), int(order[-1])):
            tok, slot = torch.nonzero(ids_c == e, as_tuple=True)
            n = tok.numel()
            assert n > 0
            r = oracle.bwd(dout[tok.cuda()].cpu(), x[tok.cuda()].cpu(), torch.zeros(n, 1, dtype=torch.int32),
                           w_c[tok, slot][:, None], W1[e:e + 1].cpu(), W2[e:e + 1].cpu())
            assert_close_bf16(dW1[e], r[1][0], f"cfg4 {what} dW_gate_up[{e}] ({n} rows)")
            assert_close_bf16(dW2[e], r[2][0], f"cfg4 {what} dW_down[{e}] ({n} rows)")

    # 1. the persistent launches against the oracle, before any other layer has written anything
    check_against_oracle(out, dx, dW1, dW2, dw, "persistent launch")
    sums = [t.view(torch.int16).to(torch.int64).sum().item() for t in (out, dx, dW1, dW2)]
    dw_fused = dw.clone()
    # 2. the operator-by-operator launches into the SAME gradient tensors (45 GB: no room for a second set), zeroed
    # first so that nothing of the persistent launches' results can pass for theirs
    for t in (dx, dW1, dW2, dw):
        t.zero_()
    assert dx.view(torch.int16).to(torch.int64).abs().sum().item() == 0
    other = MoeLayer(cfg.T, cfg.d, cfg.E, cfg.k, cfg.S, cfg.F, renorm=cfg.renorm, save_for_bwd=True, serial=True)
    out2 = other.ffn_fwd(x, ids, w, W1, W2)
    other.ffn_bwd(dout, x, ids, w, W1, W2, dx=dx, dW_gate_up=dW1, dW_down=dW2, d_topk_w=dw)
    torch.cuda.synchronize()
    assert other.status() == (0, 0)
    check_against_oracle(out2, dx, dW1, dW2, dw, "operator launches")
    # 3. both launch modes give the same bits (checksums of the four large tensors, d_topk_w in full)
    sums2 = [t.view(torch.int16).to(torch.int64).sum().item() for t in (out2, dx, dW1, dW2)]
    assert sums == sums2, "fused and serial launches disagree"
    assert torch.equal(out, out2) and torch.equal(dw, dw_fused)
    other.close()
    layer.close()
