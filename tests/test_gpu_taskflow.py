"""The descriptor runtime (Section 4.4) executing graphs compiled by the taskflow front end (Section 4.2, 4.3): the
SwiGLU + Add pair of Section 6, the same pair with an unsplit fallback, a diamond, and a chain in the opposite order --
all with the same device code -- against the fp64 oracle."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _bf(t):
    return t.to(torch.bfloat16)


def _run(tensors, ops, lag, host_tensors):
    from paper_2605_23764_b200 import binding as B
    plan = B.moe_taskflow_compile(tensors, ops, lag)
    slots = []
    for (r, c), h in zip(tensors, host_tensors):
        slots.append(h.to(DEV) if h is not None else torch.full((max(r, 1), c), float("nan"), dtype=torch.bfloat16, device=DEV))
    ws = torch.empty(B.moe_taskflow_workspace_bytes(plan["n_tds"], plan["n_events"], len(tensors)), dtype=torch.uint8, device=DEV)
    B.moe_taskflow_run(plan, slots, tensors, ws)
    assert B.moe_taskflow_status(ws) == (0, 0)
    first = [s.clone() for s in slots]
    for (r, c), h, s in zip(tensors, host_tensors, slots):        # a second step on the plan already in the workspace
        if h is None:
            s.fill_(float("nan"))
    B.moe_taskflow_run(plan, slots, tensors, ws, upload=False)
    assert B.moe_taskflow_status(ws) == (0, 0)
    for a, b in zip(first, slots):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    return plan, [s.cpu() for s in slots]


def _close(got, ref, name):
    err = np.abs(got.double().numpy() - ref)
    assert err.max() <= 2e-2 * np.abs(ref).max(), name
    assert err.sum() <= 5e-3 * np.abs(ref).sum(), name


@pytest.mark.parametrize("M,C,rows_a,rows_b,lag", [(300, 2048, 8, 8, 64), (5000, 2048, 8, 16, 4736), (1231, 1000, 4, 4, 0),
                                                   (96, 64, 32, 8, 8), (1, 8, 8, 8, 0)])
def test_swiglu_add_pair_from_descriptors(M, C, rows_a, rows_b, lag):
    import oracle
    from paper_2605_23764_b200 import binding as B
    g = torch.Generator().manual_seed(M + C)
    x, r = _bf(torch.randn(M, 2 * C, generator=g) * 1.5), _bf(torch.randn(M, C, generator=g))
    tensors = [(M, 2 * C), (M, C), (M, C), (M, C)]
    ops = [B.tf_operator(B.MOE_TF_SWIGLU, [0], [1], rows_a, split_inputs=None),
           B.tf_operator(B.MOE_TF_ADD, [1, 2], [3], rows_b, split_inputs=[(0, 0)])]
    plan, out = _run(tensors, ops, lag, [x, None, r, None])
    s_ref, z_ref = oracle.swiglu_add(x, r)
    _close(out[1], s_ref, "s"); _close(out[3], z_ref, "z")
    # the same arithmetic as the fixed schedules of moe_sched_study: bit-equal
    s2 = torch.empty(M, C, dtype=torch.bfloat16, device=DEV); z2 = torch.empty_like(s2)
    ws = torch.empty(B.moe_sched_study_workspace_bytes(M, 8), dtype=torch.uint8, device=DEV)
    B.moe_sched_study(1, x.to(DEV), r.to(DEV), s2, z2, M, C, 8, ws)
    torch.cuda.synchronize()
    assert torch.equal(out[1].view(torch.int16), s2.cpu().view(torch.int16))
    assert torch.equal(out[3].view(torch.int16), z2.cpu().view(torch.int16))


def test_unsplit_fallback_runs_as_one_task():
    import oracle
    from paper_2605_23764_b200 import binding as B
    M, C = 200, 256
    g = torch.Generator().manual_seed(1)
    x, r = _bf(torch.randn(M, 2 * C, generator=g)), _bf(torch.randn(M, C, generator=g))
    tensors = [(M, 2 * C), (M, C), (M, C), (M, C)]
    ops = [B.tf_operator(B.MOE_TF_SWIGLU, [0], [1], 8, split_inputs=None),
           B.tf_operator(B.MOE_TF_ADD, [1, 2], [3], 8, split_inputs=[(0, 1)])]      # wants a column split: not offered
    plan, out = _run(tensors, ops, 0, [x, None, r, None])
    assert plan["op_task_num"] == [25, 1]
    s_ref, z_ref = oracle.swiglu_add(x, r)
    _close(out[3], z_ref, "z")


def test_diamond_and_reversed_chain_with_the_same_runtime():
    import oracle
    from paper_2605_23764_b200 import binding as B
    M, C = 777, 512
    g = torch.Generator().manual_seed(2)
    x, r = _bf(torch.randn(M, 2 * C, generator=g)), _bf(torch.randn(M, C, generator=g))
    # diamond: s = SwiGLU(x); z1 = s + r; z2 = z1 + s
    tensors = [(M, 2 * C), (M, C), (M, C), (M, C), (M, C)]
    ops = [B.tf_operator(B.MOE_TF_SWIGLU, [0], [1], 8, split_inputs=None),
           B.tf_operator(B.MOE_TF_ADD, [1, 2], [3], 16, split_inputs=[(0, 0)]),
           B.tf_operator(B.MOE_TF_ADD, [3, 1], [4], 16, split_inputs=[(0, 0), (1, 0)])]
    plan, out = _run(tensors, ops, 64, [x, None, r, None, None])
    s_ref, z1_ref = oracle.swiglu_add(x, r)
    _close(out[3], z1_ref, "z1"); _close(out[4], z1_ref + s_ref, "z2")
    # z2 from the kernel's own bf16 intermediates: one rounding
    z2_own = out[3].double().numpy() + out[1].double().numpy()
    assert np.all(np.abs(out[4].double().numpy() - z2_own) <= np.abs(z2_own) * 2.0 ** -8 + 1e-30)
    # reversed: y = a + b ([M, 2C]); s = SwiGLU(y)
    a, b = _bf(torch.randn(M, 2 * C, generator=g)), _bf(torch.randn(M, 2 * C, generator=g))
    tensors = [(M, 2 * C), (M, 2 * C), (M, 2 * C), (M, C)]
    ops = [B.tf_operator(B.MOE_TF_ADD, [0, 1], [2], 8, split_inputs=None),
           B.tf_operator(B.MOE_TF_SWIGLU, [2], [3], 8, split_inputs=[(0, 0)])]
    plan, out = _run(tensors, ops, 64, [a, b, None, None])
    y_ref = a.double().numpy() + b.double().numpy()
    s_ref, _ = oracle.swiglu_add(y_ref, np.zeros((M, C)))
    _close(out[2], y_ref, "y"); _close(out[3], s_ref, "s")


def test_run_refuses_descriptors_that_point_outside_the_slots():
    from paper_2605_23764_b200 import binding as B
    tensors = [(16, 128), (16, 64), (16, 64), (16, 64)]
    ops = [B.tf_operator(B.MOE_TF_SWIGLU, [0], [1], 8, split_inputs=None),
           B.tf_operator(B.MOE_TF_ADD, [1, 2], [3], 8, split_inputs=[(0, 0)])]
    plan = B.moe_taskflow_compile(tensors, ops, 0)
    slots = [torch.zeros(r, c, dtype=torch.bfloat16, device=DEV) for r, c in tensors]
    ws = torch.empty(B.moe_taskflow_workspace_bytes(plan["n_tds"], plan["n_events"], 4), dtype=torch.uint8, device=DEV)
    plan["tds"][0].outputs[0].slot = 9
    with pytest.raises(B.MoeError):
        B.moe_taskflow_run(plan, slots, tensors, ws)
    plan["tds"][0].outputs[0].slot = 1
    with pytest.raises(B.MoeError):
        B.moe_taskflow_run(plan, slots[:3] + [slots[3][:8]], tensors, ws)        # a tensor smaller than its shape
    with pytest.raises(B.MoeError):
        B.moe_taskflow_run(plan, slots, tensors, ws[:64])


def test_run_without_upload_on_a_foreign_workspace_does_nothing():
    from paper_2605_23764_b200 import binding as B
    tensors = [(64, 128), (64, 64), (64, 64), (64, 64)]
    ops = [B.tf_operator(B.MOE_TF_SWIGLU, [0], [1], 8, split_inputs=None),
           B.tf_operator(B.MOE_TF_ADD, [1, 2], [3], 8, split_inputs=[(0, 0)])]
    plan = B.moe_taskflow_compile(tensors, ops, 0)
    slots = [torch.ones(r, c, dtype=torch.bfloat16, device=DEV) for r, c in tensors]
    ws = torch.zeros(B.moe_taskflow_workspace_bytes(plan["n_tds"], plan["n_events"], 4), dtype=torch.uint8, device=DEV)
    B.moe_taskflow_run(plan, slots, tensors, ws, upload=False)          # nothing was ever uploaded here
    assert B.moe_taskflow_status(ws)[0] != 0
    assert torch.all(slots[3] == 1)                                     # no task ran
    B.moe_taskflow_run(plan, slots, tensors, ws, upload=True)
    assert B.moe_taskflow_status(ws) == (0, 0)
    other = [t.clone() for t in slots]                                  # same plan, other tensors: the upload does not cover them
    B.moe_taskflow_run(plan, other, tensors, ws, upload=False)
    assert B.moe_taskflow_status(ws)[0] != 0
