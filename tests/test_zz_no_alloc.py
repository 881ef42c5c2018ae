"""The allocation-free dispatch-layout entry point (for callers that may not cudaMalloc, e.g. code
inside a pre-planned memory region or a serving loop, and callers without a context) must give
exactly what moe_layout gives -- also on a second call, which reuses the library's fixed scratch
array with the first call's contents still in it.  This file sorts last so that the rest of the
suite has already run if it fails."""
import pytest
import torch

from paper_2605_23764_b200 import MoeError, MoeLayer, binding

pytestmark = pytest.mark.gpu


def _both(T, E, k, S, seed):
    g = torch.Generator().manual_seed(seed)
    ids = torch.stack([torch.randperm(E, generator=g)[:k] for _ in range(T)]).to(torch.int32).cuda()
    layer = MoeLayer(T, 64, E, k, S, 64)
    want = layer.layout(ids)
    layer.close()
    n, Ep = T * (k + S), E + S
    i32 = dict(dtype=torch.int32, device="cuda")
    got = (torch.full((Ep,), -7, **i32), torch.full((Ep + 1,), -7, **i32), torch.full((n,), -7, **i32),
           torch.full((n,), -7, **i32))
    status = torch.full((2,), -7, **i32)
    binding.moe_layout_noalloc(ids, T, E, k, S, *got, status)
    torch.cuda.synchronize()
    for a, b, name in zip(got, want, ("counts", "offsets", "row_of", "src_of")):
        assert torch.equal(a, b), name   # integer work: bit-exact, the tolerance of the layout tests
    assert status.tolist() == [0, 0]


def test_noalloc_layout_matches_moe_layout_on_two_calls_in_a_row():
    _both(T=3000, E=64, k=6, S=2, seed=1)     # first call (sets up the scratch address on this device)
    _both(T=517, E=200, k=8, S=0, seed=2)     # second call: other sizes, scratch holds stale contents
    _both(T=3000, E=64, k=6, S=2, seed=1)     # and the first problem again


def test_noalloc_layout_reports_bad_ids_and_rejects_oversize():
    T, E, k = 64, 8, 2
    ids = torch.randint(0, E, (T, k), dtype=torch.int32)
    ids[5, 1] = 77
    i32 = dict(dtype=torch.int32, device="cuda")
    out = (torch.empty(E, **i32), torch.empty(E + 1, **i32), torch.empty(T * k, **i32), torch.empty(T * k, **i32))
    status = torch.zeros(2, **i32)
    binding.moe_layout_noalloc(ids.cuda(), T, E, k, 0, *out, status)
    torch.cuda.synchronize()
    assert status.tolist() == [1, 5 * k + 1] and out[2][5 * k + 1].item() == -1
    binding.moe_layout_noalloc(ids.clamp(0, E - 1).cuda(), T, E, k, 0, *out, status)  # status starts clean again
    torch.cuda.synchronize()
    assert status.tolist() == [0, 0]
    big_T = 262144 // k + 1
    with pytest.raises(MoeError, match="fixed limit"):
        binding.moe_layout_noalloc(ids.cuda(), big_T, E, k, 0, *out, status)
