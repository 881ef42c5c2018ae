"""SwiGLU + Add operator pair of the scheduling microbenchmarks (Section 6.1, 6.2): the three schedules
against the fp64 oracle, element by element, and against one another bit for bit."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _inputs(M, C, seed):
    g = torch.Generator().manual_seed(seed)
    x = (torch.randn(M, 2 * C, generator=g) * 1.5).to(torch.bfloat16)
    r = torch.randn(M, C, generator=g).to(torch.bfloat16)
    return x, r


def _run(mode, x, r, M, C, tile_rows):
    from paper_2605_23764_b200 import binding as B
    dev = torch.device("cuda:0")
    xd, rd = x.to(dev), r.to(dev)
    s = torch.full((max(M, 1), C), float("nan"), dtype=torch.bfloat16, device=dev)
    z = torch.full((max(M, 1), C), float("nan"), dtype=torch.bfloat16, device=dev)
    ws = torch.empty(B.moe_sched_study_workspace_bytes(M, tile_rows), dtype=torch.uint8, device=dev)
    B.moe_sched_study(mode, xd, rd, s, z, M, C, tile_rows, ws)
    status, ns, tasks = B.moe_sched_study_stats(ws)
    assert status == (0, 0)
    return s[:M].cpu(), z[:M].cpu(), ns, tasks


@pytest.mark.parametrize("M,C,tile_rows", [(1, 8, 1), (37, 64, 4), (300, 2048, 8), (2048, 2048, 8), (5000, 2048, 16),
                                           (1231, 1000, 3)])
def test_three_schedules_match_the_oracle(M, C, tile_rows):
    import oracle
    x, r = _inputs(M, C, 100 + M)
    s_ref, z_ref = oracle.swiglu_add(x.double().numpy(), r.double().numpy())
    outs = []
    for mode in (0, 1, 2):
        s, z, ns, tasks = _run(mode, x, r, M, C, tile_rows)
        ntiles = -(-M // tile_rows)
        assert tasks == (0 if mode == 0 else 2 * ntiles)
        # s is one bf16 rounding of an fp32 evaluation of the fp64 value; z adds one more rounding on top of bf16(s)
        for got, ref, name in ((s, s_ref, "s"), (z, z_ref, "z")):
            err = np.abs(got.double().numpy() - ref)
            scale = np.abs(ref).max()
            assert err.max() <= 2e-2 * scale, (name, mode, err.max(), scale)
            assert err.sum() <= 5e-3 * np.abs(ref).sum(), (name, mode)
        # z against the oracle applied to the kernel's own bf16 intermediate: one rounding only
        z_from_s = s.double().numpy() + r.double().numpy()
        assert np.all(np.abs(z.double().numpy() - z_from_s) <= np.abs(z_from_s) * 2.0 ** -8 + 1e-30)
        outs.append((s, z))
    for s, z in outs[1:]:
        assert torch.equal(s.view(torch.int16), outs[0][0].view(torch.int16))
        assert torch.equal(z.view(torch.int16), outs[0][1].view(torch.int16))


def test_empty_input_launches_nothing():
    x, r = _inputs(1, 64, 5)
    for mode in (0, 1, 2):
        s, z, ns, tasks = _run(mode, x[:0].reshape(0, 128), r[:0].reshape(0, 64), 0, 64, 8)
        assert tasks == 0 and s.numel() == 0


def test_rejects_bad_arguments():
    from paper_2605_23764_b200 import binding as B
    dev = torch.device("cuda:0")
    x = torch.zeros(16, 128, dtype=torch.bfloat16, device=dev)
    r = torch.zeros(16, 64, dtype=torch.bfloat16, device=dev)
    s, z = torch.zeros_like(r), torch.zeros_like(r)
    ws = torch.empty(B.moe_sched_study_workspace_bytes(16, 4), dtype=torch.uint8, device=dev)
    with pytest.raises(B.MoeError):
        B.moe_sched_study(3, x, r, s, z, 16, 64, 4, ws)          # unknown mode
    with pytest.raises(B.MoeError):
        B.moe_sched_study(1, x, r, s, z, 16, 60, 4, ws)          # C % 8 != 0
    with pytest.raises(B.MoeError):
        B.moe_sched_study(1, x, r, s, z, 16, 64, 4, ws[:64])     # workspace too small
    with pytest.raises(B.MoeError):
        B.moe_sched_study(1, x, r, s, z, 32, 64, 4, ws)          # tensors smaller than M rows
