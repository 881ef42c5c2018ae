"""Token-column tiles at their edges: experts whose token counts sit on and around the 32-token grain,
the 128-row M-block and the 256-token tile, through forward and backward in both launch modes."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_23764_b200 import MoeLayer
from tests.gpu_util import assert_close_bf16

pytestmark = pytest.mark.gpu

# rows per expert: empty, one token, around 32, around one M-block, around one 256-token tile (one unit of two
# M-blocks vs a single block followed by block + tail), three and five M-blocks, a long expert
COUNTS = [0, 1, 31, 32, 33, 127, 128, 129, 160, 255, 256, 257, 300, 383, 384, 385, 513, 640, 1100, 0, 5]


def _problem(d, F, seed):
    counts = np.array(COUNTS)
    E, T = len(counts), int(counts.sum())
    g = torch.Generator().manual_seed(seed)
    ids = torch.from_numpy(np.repeat(np.arange(E), counts).astype(np.int32))
    ids = ids[torch.randperm(T, generator=g)].reshape(T, 1).contiguous()
    w = (torch.rand(T, 1, generator=g) + 0.25).float()
    x = torch.randn(T, d, generator=g).to(torch.bfloat16)
    W1 = (torch.randn(E, 2 * F, d, generator=g) / d ** 0.5).to(torch.bfloat16)
    W2 = (torch.randn(E, d, F, generator=g) / d ** 0.5).to(torch.bfloat16)
    dout = torch.randn(T, d, generator=g).to(torch.bfloat16)
    return T, E, [t.cuda() for t in (ids, w, x, W1, W2, dout)]


@pytest.mark.parametrize("d,F", [(192, 80), (320, 256)])
@pytest.mark.parametrize("serial", [False, True])
def test_counts_on_tile_edges(d, F, serial):
    T, E, (ids, w, x, W1, W2, dout) = _problem(d, F, seed=d + F)
    layer = MoeLayer(T, d, E, 1, 0, F, renorm=False, save_for_bwd=True, serial=serial)
    out = layer.ffn_fwd(x, ids, w, W1, W2)
    dx, dW1, dW2, dw = layer.ffn_bwd(dout, x, ids, w, W1, W2)
    torch.cuda.synchronize()
    assert layer.status() == (0, 0)
    ref_out = oracle.fwd(x, ids.cpu(), w.cpu(), W1, W2)
    rdx, rdW1, rdW2, rdw = oracle.bwd(dout, x, ids.cpu(), w.cpu(), W1, W2)
    assert_close_bf16(out, ref_out, "out")
    assert_close_bf16(dx, rdx, "dx")
    assert_close_bf16(dW1, rdW1, "dW_gate_up")
    assert_close_bf16(dW2, rdW2, "dW_down")
    assert_close_bf16(dw, rdw, "d_topk_w")
    # every expert on its own, at the same tolerance as the whole tensors: a wrong tile edge would hide in
    # whole-tensor norms
    ref_out, rdx = np.asarray(ref_out), np.asarray(rdx)
    for e, n in enumerate(COUNTS):
        if n == 0:
            assert torch.count_nonzero(dW1[e]).item() == 0 and torch.count_nonzero(dW2[e]).item() == 0
        else:
            tok = (ids[:, 0] == e).nonzero()[:, 0].cpu()
            assert_close_bf16(dW2[e], rdW2[e], f"dW_down[{e}] ({n} tokens)")
            assert_close_bf16(dW1[e], rdW1[e], f"dW_gate_up[{e}] ({n} tokens)")
            assert_close_bf16(out[tok], ref_out[tok.numpy()], f"out of expert {e} ({n} tokens)")
            assert_close_bf16(dx[tok], rdx[tok.numpy()], f"dx of expert {e} ({n} tokens)")
            assert_close_bf16(dw[tok], np.asarray(rdw)[tok.numpy()], f"d_topk_w of expert {e} ({n} tokens)")
    layer.close()


def _check_against_oracle(T, d, E, k, F, ids, w, seed, serial):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(T, d, generator=g).to(torch.bfloat16).cuda()
    W1 = (torch.randn(E, 2 * F, d, generator=g) / d ** 0.5).to(torch.bfloat16).cuda()
    W2 = (torch.randn(E, d, F, generator=g) / d ** 0.5).to(torch.bfloat16).cuda()
    dout = torch.randn(T, d, generator=g).to(torch.bfloat16).cuda()
    layer = MoeLayer(T, d, E, k, 0, F, renorm=False, save_for_bwd=True, serial=serial)
    out = layer.ffn_fwd(x, ids, w, W1, W2)
    dx, dW1, dW2, dw = layer.ffn_bwd(dout, x, ids, w, W1, W2)
    torch.cuda.synchronize()
    assert layer.status() == (0, 0)
    ref_out = oracle.fwd(x, ids.cpu(), w.cpu(), W1, W2)
    rdx, rdW1, rdW2, rdw = oracle.bwd(dout, x, ids.cpu(), w.cpu(), W1, W2)
    for got, ref, name in ((out, ref_out, "out"), (dx, rdx, "dx"), (dW1, rdW1, "dW_gate_up"), (dW2, rdW2, "dW_down"),
                           (dw, rdw, "d_topk_w")):
        assert_close_bf16(got, ref, name)
    counts = np.bincount(ids.cpu().numpy().reshape(-1), minlength=E)
    for e in np.nonzero(counts == 0)[0]:
        assert torch.count_nonzero(dW1[e]).item() == 0 and torch.count_nonzero(dW2[e]).item() == 0
    layer.close()


@pytest.mark.parametrize("serial", [False, True])
def test_every_token_to_one_expert(serial):
    """The degenerate routing: one expert holds all 1000 rows (eight M-blocks), the other seven none."""
    T, d, E, F = 1000, 128, 8, 96
    ids = torch.full((T, 1), 5, dtype=torch.int32).cuda()
    w = torch.linspace(0.1, 1.0, T).reshape(T, 1).float().cuda()
    _check_against_oracle(T, d, E, 1, F, ids, w, 11, serial)


@pytest.mark.parametrize("serial", [False, True])
def test_top_k_equals_number_of_experts(serial):
    """k = E: every expert receives every token."""
    T, d, E, F = 300, 128, 4, 64
    g = torch.Generator().manual_seed(5)
    ids = torch.stack([torch.randperm(E, generator=g) for _ in range(T)]).to(torch.int32).cuda()
    w = torch.softmax(torch.randn(T, E, generator=g), dim=1).float().cuda()
    _check_against_oracle(T, d, E, E, F, ids, w, 12, serial)


@pytest.mark.parametrize("serial", [False, True])
def test_more_experts_than_rows(serial):
    """E > T k: at most six of the 64 experts hold a row."""
    T, d, E, k, F = 3, 64, 64, 2, 32
    ids = torch.tensor([[7, 40], [40, 63], [0, 7]], dtype=torch.int32).cuda()
    w = torch.tensor([[0.7, 0.3], [0.5, 0.5], [0.9, 0.1]]).float().cuda()
    _check_against_oracle(T, d, E, k, F, ids, w, 13, serial)


def test_wide_rows_take_the_bulk_copy_gather():
    """Rows of 8 KB and more are gathered with bulk copies (whole rows through shared-memory slots, padding
    rows from a zeroed slot): d = 4096 with ragged expert segments, forward and backward."""
    T, d, E, k, F = 700, 4096, 6, 2, 32
    g = torch.Generator().manual_seed(3)
    ids = torch.stack([torch.randperm(E, generator=g)[:k] for _ in range(T)]).to(torch.int32).cuda()
    w = torch.softmax(torch.randn(T, k, generator=g), dim=1).float().cuda()
    _check_against_oracle(T, d, E, k, F, ids, w, 14, serial=True)


@pytest.mark.parametrize("serial", [False, True])
def test_skewed_routing_forward_and_backward(serial):
    """Zipf-like expert popularity with four unreachable experts: segments from empty to a few thousand rows
    (streamed and resident weight-gradient strips, token tiles of one and two M-blocks side by side)."""
    T, d, E, k, F = 2048, 512, 32, 4, 256
    g = torch.Generator().manual_seed(21)
    rank = torch.randperm(E, generator=g).float()
    logits = torch.randn(T, E, generator=g) * 1.3 - 1.2 * torch.log(rank + 1.0)
    logits[:, rank >= E - 4] = -1e4
    top = torch.topk(logits, k, dim=1)
    ids = top.indices.to(torch.int32).cuda()
    w = torch.softmax(top.values, dim=1).float().cuda()
    counts = np.bincount(ids.cpu().numpy().reshape(-1), minlength=E)
    assert (counts == 0).sum() >= 4 and counts.max() > 640, counts
    _check_against_oracle(T, d, E, k, F, ids, w, 22, serial)
