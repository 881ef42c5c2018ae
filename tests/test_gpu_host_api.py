"""The host-buffer entry points (pinned host activations in, host results out) and the per-operator
timing calls give the same results as the device-buffer calls."""
import pytest
import torch

from paper_2605_23764_b200 import MoeLayer, binding as B
from tests.gpu_util import small_problem

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("serial", [False, True])
def test_host_buffer_calls_match_device_calls(serial):
    T, d, E, k, S, F = 333, 192, 12, 3, 1, 160
    x, W1, W2, logits, dout = small_problem(T, d, E, k, S, F, 21)
    layer = MoeLayer(T, d, E, k, S, F, renorm=True, save_for_bwd=True, serial=serial)
    ids, w = layer.route(logits)
    out = layer.ffn_fwd(x, ids, w, W1, W2)
    dx, dW1, dW2, dw = layer.ffn_bwd(dout, x, ids, w, W1, W2)
    torch.cuda.synchronize()

    pin = dict(pin_memory=True)
    lh, xh, doh = logits.cpu().pin_memory(), x.cpu().pin_memory(), dout.cpu().pin_memory()
    idh = torch.empty(T, k, dtype=torch.int32, **pin)
    wh = torch.empty(T, k, dtype=torch.float32, **pin)
    oh = torch.empty(T, d, dtype=torch.bfloat16, **pin)
    dxh = torch.empty(T, d, dtype=torch.bfloat16, **pin)
    dwh = torch.empty(T, k, dtype=torch.float32, **pin)
    dW1b, dW2b = torch.empty_like(W1), torch.empty_like(W2)
    B.moe_route_host(layer.ctx, lh, T, idh, wh)
    B.moe_ffn_fwd_host(layer.ctx, xh, idh, wh, W1, W2, oh, T)
    B.moe_ffn_bwd_host(layer.ctx, doh, W1, W2, dxh, dW1b, dW2b, dwh, T)
    torch.cuda.synchronize()
    assert layer.status() == (0, 0)
    assert torch.equal(idh, ids.cpu()) and torch.equal(wh, w.cpu())
    assert torch.equal(oh, out.cpu()) and torch.equal(dxh, dx.cpu()) and torch.equal(dwh, dw.cpu())
    assert torch.equal(dW1b, dW1) and torch.equal(dW2b, dW2)
    layer.close()


def test_phase_times_are_reported_per_operator():
    T, d, E, k, S, F = 512, 256, 8, 2, 0, 256
    x, W1, W2, logits, dout = small_problem(T, d, E, k, S, F, 5)
    for serial, want in ((True, {"layout", "gather", "gemm_gate_up", "gemm_down", "combine"}),
                         (False, {"layout", "fused_fwd"})):
        layer = MoeLayer(T, d, E, k, S, F, serial=serial)
        ids, w = layer.route(logits)
        B.moe_set_profiling(layer.ctx, True)
        layer.ffn_fwd(x, ids, w, W1, W2)
        ph = B.moe_get_phase_ms(layer.ctx)
        assert set(ph) == want and all(v > 0 for v in ph.values())
        assert layer.launches() == (7 if serial else 5)   # layout x3 + the four operators, or layout x3 + combine order + the one persistent launch
        layer.close()


@pytest.mark.parametrize("serial", [False, True])
def test_back_to_back_host_steps_keep_their_own_inputs(serial):
    """Three training steps through the host entry points with different inputs and no synchronisation in
    between: the copy-in stream may run ahead of the compute stream, so a step's x / dout must not land in
    the staging buffers before the previous step has read them."""
    T, d, E, k, S, F = 1500, 256, 8, 2, 0, 128   # T >= 256: the chunked copy-out of the forward is in play
    pin = dict(pin_memory=True)
    layer = MoeLayer(T, d, E, k, S, F, renorm=True, save_for_bwd=True, serial=serial)
    ref = MoeLayer(T, d, E, k, S, F, renorm=True, save_for_bwd=True, serial=serial)
    steps = []
    for i in range(3):
        x, W1, W2, logits, dout = small_problem(T, d, E, k, S, F, 100 + i)
        ids, w = ref.route(logits)
        out = ref.ffn_fwd(x, ids, w, W1, W2)
        dx, dW1, dW2, dw = ref.ffn_bwd(dout, x, ids, w, W1, W2)
        steps.append(dict(x=x.cpu().pin_memory(), dout=dout.cpu().pin_memory(), ids=ids.cpu().pin_memory(),
                          w=w.cpu().pin_memory(), W1=W1, W2=W2, out=out.cpu(), dx=dx.cpu(), dw=dw.cpu(),
                          dW1=dW1.clone(), dW2=dW2.clone(),
                          oh=torch.empty(T, d, dtype=torch.bfloat16, **pin),
                          dxh=torch.empty(T, d, dtype=torch.bfloat16, **pin),
                          dwh=torch.empty(T, k, dtype=torch.float32, **pin),
                          gW1=torch.empty_like(W1), gW2=torch.empty_like(W2)))
    torch.cuda.synchronize()
    for s in steps:   # enqueue everything, synchronise once
        B.moe_ffn_fwd_host(layer.ctx, s["x"], s["ids"], s["w"], s["W1"], s["W2"], s["oh"], T)
        B.moe_ffn_bwd_host(layer.ctx, s["dout"], s["W1"], s["W2"], s["dxh"], s["gW1"], s["gW2"], s["dwh"], T)
    torch.cuda.synchronize()
    assert layer.status() == (0, 0)
    for i, s in enumerate(steps):
        assert torch.equal(s["oh"], s["out"]), f"step {i}: out"
        assert torch.equal(s["dxh"], s["dx"]), f"step {i}: dx"
        assert torch.equal(s["dwh"], s["dw"]), f"step {i}: d_topk_w"
        assert torch.equal(s["gW1"], s["dW1"]) and torch.equal(s["gW2"], s["dW2"]), f"step {i}: weight gradients"
    layer.close()
    ref.close()


@pytest.mark.parametrize("serial", [False, True])
def test_deferred_out_copy_is_complete_after_the_backward_call(serial):
    """MOE_FLAG_DEFER_OUT_COPY: the forward result leaves behind the backward; after the backward call's stream work it
    is there, the step's other results are unchanged, and back-to-back steps keep their own results."""
    T, d, E, k, S, F = 700, 256, 12, 3, 0, 160
    x, W1, W2, logits, dout = small_problem(T, d, E, k, S, F, 33)
    ref = MoeLayer(T, d, E, k, S, F, renorm=True, save_for_bwd=True, serial=serial)
    ids, w = ref.route(logits)
    out = ref.ffn_fwd(x, ids, w, W1, W2).clone()
    dx, dW1, dW2, dw = [t.clone() for t in ref.ffn_bwd(dout, x, ids, w, W1, W2)]
    out2 = ref.ffn_fwd((x.float() * 0.5).to(torch.bfloat16), ids, w, W1, W2).clone()
    torch.cuda.synchronize()
    ref.close()
    layer = MoeLayer(T, d, E, k, S, F, renorm=True, save_for_bwd=True, serial=serial, defer_out_copy=True)
    pin = dict(pin_memory=True)
    xh, x2h, doh = x.cpu().pin_memory(), (x.float() * 0.5).to(torch.bfloat16).cpu().pin_memory(), dout.cpu().pin_memory()
    idh, wh = ids.cpu().pin_memory(), w.cpu().pin_memory()
    oh = torch.full((T, d), float("nan"), dtype=torch.bfloat16).pin_memory()
    oh2 = torch.full((T, d), float("nan"), dtype=torch.bfloat16).pin_memory()
    dxh = torch.empty(T, d, dtype=torch.bfloat16, **pin)
    dwh = torch.empty(T, k, dtype=torch.float32, **pin)
    gW1, gW2 = torch.empty_like(W1), torch.empty_like(W2)
    B.moe_ffn_fwd_host(layer.ctx, xh, idh, wh, W1, W2, oh, T)
    B.moe_ffn_bwd_host(layer.ctx, doh, W1, W2, dxh, gW1, gW2, dwh, T)
    B.moe_ffn_fwd_host(layer.ctx, x2h, idh, wh, W1, W2, oh2, T)        # the next step reuses the staging buffer
    torch.cuda.current_stream().synchronize()
    assert torch.equal(oh, out.cpu()) and torch.equal(dxh, dx.cpu()) and torch.equal(dwh, dw.cpu())
    assert torch.equal(gW1, dW1) and torch.equal(gW2, dW2)
    assert layer.status() == (0, 0)                                      # also completes the second forward's copy
    assert torch.equal(oh2, out2.cpu())
    layer.close()
