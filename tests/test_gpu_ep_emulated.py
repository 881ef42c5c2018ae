"""Expert-parallel Dispatch / Combine with one-sided put + signal (Section 4.1, Section 4.5), all ranks emulated on ONE
GPU: every rank's buffers live on the device and one cooperative launch plays the producers and consumers of every rank.
Integer and copied data are compared bit for bit with the oracle; the composed layer (dispatch -> each rank's experts ->
combine) is compared with the oracle's single-device layer and must be bit-equal to this library's single-device layer."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _problem(R, E, k, d, F, Ts, seed):
    g = torch.Generator().manual_seed(seed)
    x = [torch.randn(T, d, generator=g).to(torch.bfloat16) for T in Ts]
    logits = [torch.randn(T, E, generator=g) for T in Ts]
    W1 = (torch.randn(E, 2 * F, d, generator=g) / d ** 0.5).to(torch.bfloat16)
    W2 = (torch.randn(E, d, F, generator=g) / F ** 0.5).to(torch.bfloat16)
    return x, logits, W1, W2


@pytest.mark.parametrize("R,E,k,d,F,Ts", [(2, 8, 2, 256, 128, [300, 77]), (4, 16, 3, 192, 64, [64, 0, 500, 129]),
                                          (8, 64, 6, 512, 128, [256] * 8)])
def test_emulated_ranks_dispatch_compute_combine(R, E, k, d, F, Ts):
    import oracle
    from oracle import ep_oracle
    from paper_2605_23764_b200 import MoeLayer, binding as B
    El = E // R
    x, logits, W1, W2 = _problem(R, E, k, d, F, Ts, 17 * R + E)
    i32 = dict(dtype=torch.int32, device=DEV)
    status = torch.zeros(4, **i32)

    # ---- per rank: routing and the local expert-ordered layout (over all E experts), as the single-device path does
    ids, w, src_of, counts = [], [], [], []
    for s in range(R):
        lay = MoeLayer(max(Ts[s], 1), d, E, k, 0, F, renorm=True)
        if Ts[s]:
            i_s, w_s = lay.route(logits[s].to(DEV))
            c = torch.empty(E, **i32); o = torch.empty(E + 1, **i32); ro = torch.empty(Ts[s] * k, **i32); so = torch.empty(Ts[s] * k, **i32)
            B.moe_layout(lay.ctx, i_s, Ts[s], c, o, ro, so)
            torch.cuda.synchronize()
        else:
            i_s, w_s = torch.empty(0, k, **i32), torch.empty(0, k, dtype=torch.float32, device=DEV)
            c, so = torch.zeros(E, **i32), torch.empty(0, **i32)
        ids.append(i_s.clone()); w.append(w_s.clone()); src_of.append(so.clone()); counts.append(c.cpu().numpy())
        lay.close()
    counts = np.stack(counts).astype(np.int32)                     # the all-gathered metadata

    # ---- plans and buffers
    plans = [B.moe_ep_plan(counts, s) for s in range(R)]
    recv_rows = plans[0][1]
    recv = [torch.full((max(int(n), 1), d), float("nan"), dtype=torch.bfloat16, device=DEV) for n in recv_rows]
    meta = [torch.full((max(int(n), 1), 4), -1, **i32) for n in recv_rows]
    rcnt = [torch.full((max(-(-int(n) // B.MOE_EP_BLOCK_ROWS), 1),), 12345, **i32) for n in recv_rows]   # stale: the call clears
    ret = [torch.full((max(T * k, 1), d), float("nan"), dtype=torch.bfloat16, device=DEV) for T in Ts]
    tcnt = [torch.full((max(-(-T // B.MOE_EP_TOKEN_BLOCK), 1),), 777, **i32) for T in Ts]
    peers = [B.moe_ep_peer(recv[q], meta[q], rcnt[q], ret[q], tcnt[q]) for q in range(R)]
    consumed = [torch.full_like(recv[q], float("nan")) for q in range(R)]
    tickets = [torch.zeros(2, **i32) for _ in range(R)]
    xs = [t.to(DEV) for t in x]
    tasks_dev = [torch.from_numpy(plans[s][0]).to(DEV) if len(plans[s][0]) else None for s in range(R)]
    locals_ = [dict(rank=s, T=Ts[s], x=xs[s], topk_w=w[s], src_of=src_of[s], tasks=tasks_dev[s], recv_rows=int(recv_rows[s]),
                    consumed=consumed[s], ticket=tickets[s]) for s in range(R)]
    B.moe_ep_dispatch(peers, locals_, k, d, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[:2] == [0, 0]

    # ---- Dispatch against the oracle: rows, meta and what the consumers read are bit-exact; counters at their thresholds
    ref = ep_oracle.ep_dispatch([t.float().numpy() for t in x], [i.cpu().numpy() for i in ids], [t.cpu().numpy() for t in w], E)
    thr = ep_oracle.ep_arrival_counts([i.cpu().numpy() for i in ids], E, B.MOE_EP_BLOCK_ROWS)
    for q in range(R):
        n = int(recv_rows[q])
        assert n == ref[q]["rows"].shape[0]
        np.testing.assert_array_equal(recv[q][:n].float().cpu().numpy(), ref[q]["rows"])
        np.testing.assert_array_equal(consumed[q][:n].float().cpu().numpy(), ref[q]["rows"])
        m = meta[q][:n].cpu().numpy()
        np.testing.assert_array_equal(m[:, :2], ref[q]["meta"])
        np.testing.assert_array_equal(m[:, 2].view(np.float32), ref[q]["w"].astype(np.float32))
        np.testing.assert_array_equal(rcnt[q][:len(thr[q])].cpu().numpy(), thr[q])

    # ---- each rank's experts on the rows it received (a k = 1 problem for the single-device layer)
    y = []
    for q in range(R):
        n = int(recv_rows[q])
        if n == 0:
            y.append(torch.empty(1, d, dtype=torch.bfloat16, device=DEV)); continue
        offs = plans[q][2]
        eid = torch.repeat_interleave(torch.arange(El, dtype=torch.int32), torch.from_numpy(np.diff(offs)).long()).reshape(n, 1).to(DEV)
        wq = meta[q][:n, 2].contiguous().view(torch.float32).reshape(n, 1).contiguous()
        lay = MoeLayer(n, d, El, 1, 0, F)
        y.append(lay.ffn_fwd(recv[q][:n].contiguous(), eid, wq, W1[q * El:(q + 1) * El].contiguous().to(DEV),
                             W2[q * El:(q + 1) * El].contiguous().to(DEV)).clone())
        assert lay.status() == (0, 0)
        lay.close()

    # ---- Combine
    out = [torch.full((max(T, 1), d), float("nan"), dtype=torch.bfloat16, device=DEV) for T in Ts]
    locals_c = [dict(rank=s, T=Ts[s], recv_rows=int(recv_rows[s]), y=y[s], out=out[s], ticket=tickets[s]) for s in range(R)]
    B.moe_ep_combine(peers, locals_c, k, d, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[:2] == [0, 0]
    for s in range(R):
        nb = -(-Ts[s] // B.MOE_EP_TOKEN_BLOCK)
        want = [min(B.MOE_EP_TOKEN_BLOCK, Ts[s] - b * B.MOE_EP_TOKEN_BLOCK) * k for b in range(nb)]
        assert tcnt[s][:nb].cpu().tolist() == want

    # ---- the whole layer: against the oracle on the ranks' tokens laid end to end, and bit-equal to the single-device path
    xg = torch.cat(x); idg = torch.cat([i.cpu() for i in ids]); wg = torch.cat([t.cpu() for t in w])
    got = torch.cat([out[s][:Ts[s]].cpu() for s in range(R)])
    ref_out = oracle.fwd(xg, idg, wg, W1, W2)
    err = np.abs(got.double().numpy() - ref_out)
    assert err.max() <= 2e-2 * np.abs(ref_out).max() and err.sum() <= 5e-3 * np.abs(ref_out).sum()
    lay = MoeLayer(sum(Ts), d, E, k, 0, F)
    single = lay.ffn_fwd(xg.to(DEV), idg.to(DEV), wg.to(DEV), W1.to(DEV), W2.to(DEV)).cpu()
    lay.close()
    assert torch.equal(got.view(torch.int16), single.view(torch.int16))


def test_dispatch_refuses_bad_arguments():
    from paper_2605_23764_b200 import binding as B
    i32 = dict(dtype=torch.int32, device=DEV)
    z = torch.zeros(8, **i32)
    bf = torch.zeros(8, 64, dtype=torch.bfloat16, device=DEV)
    peers = [B.moe_ep_peer(bf, torch.zeros(8, 4, **i32), z, bf, z)]
    loc = [dict(rank=0, T=8, x=bf, topk_w=torch.zeros(8, 1, device=DEV), src_of=z, tasks=None, recv_rows=8, consumed=None,
                ticket=torch.zeros(2, **i32))]
    with pytest.raises(B.MoeError):
        B.moe_ep_dispatch(peers, loc, 1, 60, torch.zeros(4, **i32))               # d % 8 != 0
    loc[0]["rank"] = 3
    with pytest.raises(B.MoeError):
        B.moe_ep_dispatch(peers, loc, 1, 64, torch.zeros(4, **i32))               # rank outside the peer table
