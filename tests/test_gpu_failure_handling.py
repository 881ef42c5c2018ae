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
