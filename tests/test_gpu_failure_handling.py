"""Bounded device-side waits: a dependency that is never satisfied must end the persistent launch
with MOE_ERR_TIMEOUT after the wait budget -- the kernel returns normally, nothing traps or hangs --
and the context must work again afterwards."""
import time

import pytest
import torch

import oracle
from paper_2605_23764_b200 import MoeLayer, binding
from tests.gpu_util import assert_close_bf16, small_problem

pytestmark = pytest.mark.gpu

SITE_DEP = 5


def test_unreachable_dependency_times_out_and_context_recovers():
    T, d, E, k, S, F = 256, 256, 8, 2, 0, 128
    x, W1, W2, logits, _ = small_problem(T, d, E, k, S, F, 11)
    layer = MoeLayer(T, d, E, k, S, F)
    ids, w = layer.route(logits)
    good = layer.ffn_fwd(x, ids, w, W1, W2).clone()
    assert layer.status() == (0, 0)

    binding.moe_set_wait_budget_ms(layer.ctx, 100)
    binding.moe_debug_set_unreachable_dependency(layer.ctx, True)
    t0 = time.perf_counter()
    layer.ffn_fwd(x, ids, w, W1, W2)
    code, detail = layer.status()          # synchronises: the launch has ended by itself
    elapsed = time.perf_counter() - t0
    assert code == 2, (code, detail)       # MOE_ERR_TIMEOUT
    # the scheduler's dependency poll and the roles idling behind it run out at about the same time;
    # whichever reports first names its own wait site
    assert (detail >> 24) in (1, 2, 3, 4, SITE_DEP)
    assert elapsed < 5.0                   # budget 0.1 s per wait, not a hang

    binding.moe_debug_set_unreachable_dependency(layer.ctx, False)
    binding.moe_set_wait_budget_ms(layer.ctx, 2000)
    again = layer.ffn_fwd(x, ids, w, W1, W2)
    assert layer.status() == (0, 0)
    assert torch.equal(again, good)
    ref = oracle.fwd(x, ids.cpu(), w.cpu(), W1, W2)
    assert_close_bf16(again, ref, "forward after a timed-out launch")
    layer.close()


def test_timed_out_backward_releases_the_copy_out_stream():
    """Host-buffer backward in the persistent mode: the copy of dx waits on a word the kernel sets after its last
    combine task.  A launch that gives up never sets it; the call must still end (the word is also written behind
    the launch) and the next step must be right."""
    T, d, E, k, S, F = 256, 256, 8, 2, 0, 128
    x, W1, W2, logits, dout = small_problem(T, d, E, k, S, F, 12)
    layer = MoeLayer(T, d, E, k, S, F, save_for_bwd=True)
    ids, w = layer.route(logits)
    layer.ffn_fwd(x, ids, w, W1, W2)
    dx_good, dW1_good, dW2_good, dw_good = [t.clone() for t in layer.ffn_bwd(dout, x, ids, w, W1, W2)]
    assert layer.status() == (0, 0)

    pin = dict(pin_memory=True)
    xh, doh = x.cpu().pin_memory(), dout.cpu().pin_memory()
    idh, wh = ids.cpu().pin_memory(), w.cpu().pin_memory()
    oh = torch.empty(T, d, dtype=torch.bfloat16, **pin)
    dxh = torch.empty(T, d, dtype=torch.bfloat16, **pin)
    dwh = torch.empty(T, k, dtype=torch.float32, **pin)
    gW1, gW2 = torch.empty_like(W1), torch.empty_like(W2)

    binding.moe_ffn_fwd_host(layer.ctx, xh, idh, wh, W1, W2, oh, T)
    binding.moe_set_wait_budget_ms(layer.ctx, 100)
    binding.moe_debug_set_unreachable_dependency(layer.ctx, True)
    t0 = time.perf_counter()
    binding.moe_ffn_bwd_host(layer.ctx, doh, W1, W2, dxh, gW1, gW2, dwh, T)
    code, detail = layer.status()
    torch.cuda.synchronize()               # every stream of the context has drained
    assert code == 2, (code, detail)
    assert time.perf_counter() - t0 < 5.0

    binding.moe_debug_set_unreachable_dependency(layer.ctx, False)
    binding.moe_set_wait_budget_ms(layer.ctx, 2000)
    binding.moe_ffn_fwd_host(layer.ctx, xh, idh, wh, W1, W2, oh, T)
    binding.moe_ffn_bwd_host(layer.ctx, doh, W1, W2, dxh, gW1, gW2, dwh, T)
    torch.cuda.synchronize()
    assert layer.status() == (0, 0)
    assert torch.equal(dxh, dx_good.cpu()) and torch.equal(dwh, dw_good.cpu())
    assert torch.equal(gW1, dW1_good) and torch.equal(gW2, dW2_good)
    layer.close()
