"""Host side of the expert-parallel path (Section 4.1: Dispatch as independent remote-write tasks; Section 4.5: rank-aware
task reordering): the task list every rank derives from the all-gathered expert counts, against the oracle's Dispatch.
CPU only -- including a two-process run over gloo in which each rank knows only its own routing."""
import os
import subprocess
import sys

import numpy as np
import pytest

from oracle import ep_oracle
from paper_2605_23764_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _problem(R, E, k, d, Ts, seed):
    rng = np.random.default_rng(seed)
    x = [rng.normal(size=(T, d)) for T in Ts]
    ids = [np.array([rng.permutation(E)[:k] for _ in range(T)], dtype=np.int32).reshape(T, k) for T in Ts]
    w = [rng.uniform(0.1, 1.0, size=(T, k)) for T in Ts]
    return x, ids, w


def _local_order(ids_s, E):
    """Expert-ordered local rows of one rank (stable by slot): what moe_layout's src_of holds."""
    flat = ids_s.reshape(-1)
    return np.argsort(flat, kind="stable").astype(np.int32)


@pytest.mark.parametrize("R,E,k,Ts", [(2, 8, 2, [100, 37]), (4, 8, 3, [7, 0, 120, 5]), (8, 64, 6, [50] * 8), (1, 4, 2, [33])])
def test_executing_the_plans_reproduces_the_oracle_dispatch(R, E, k, Ts):
    d = 3
    x, ids, w = _problem(R, E, k, d, Ts, R + E)
    counts = np.stack([np.bincount(i.reshape(-1), minlength=E) for i in ids]).astype(np.int32)
    ref = ep_oracle.ep_dispatch(x, ids, w, E)
    recv = [np.full((ref[q]["rows"].shape[0], d), np.nan) for q in range(R)]
    meta = [np.full((ref[q]["rows"].shape[0], 2), -1, dtype=np.int64) for q in range(R)]
    arrivals = [np.zeros(-(-ref[q]["rows"].shape[0] // B.MOE_EP_BLOCK_ROWS), dtype=np.int64) for q in range(R)]
    for s in range(R):
        tasks, recv_rows, offs = B.moe_ep_plan(counts, s)
        assert list(recv_rows) == [ref[q]["rows"].shape[0] for q in range(R)]
        np.testing.assert_array_equal(offs, ref[s]["expert_offsets"])
        src_of = _local_order(ids[s], E)
        covered = np.zeros(Ts[s] * k, dtype=np.int64)
        if len(tasks):
            order = [int(q) for q in tasks[:, 3]]
            rot = [(q - s - 1) % R for q in order]
            assert rot == sorted(rot)                              # destinations s+1, s+2, ..., s: rank-rotated
        for e, r0, n, q, d0 in tasks:
            assert 1 <= n <= B.MOE_EP_TILE_ROWS and q == e // (E // R)
            for r in range(n):
                slot = src_of[r0 + r]
                assert ids[s].reshape(-1)[slot] == e
                covered[r0 + r] += 1
                assert np.isnan(recv[q][d0 + r, 0])               # nobody else writes this row
                recv[q][d0 + r] = x[s][slot // k]
                meta[q][d0 + r] = (s, slot)
                arrivals[q][(d0 + r) // B.MOE_EP_BLOCK_ROWS] += 1
        assert np.all(covered == 1)
    thr = ep_oracle.ep_arrival_counts(ids, E, B.MOE_EP_BLOCK_ROWS)
    for q in range(R):
        np.testing.assert_array_equal(recv[q], ref[q]["rows"])
        np.testing.assert_array_equal(meta[q], ref[q]["meta"])
        np.testing.assert_array_equal(arrivals[q], thr[q])


def test_plan_rejects_bad_arguments():
    c = np.ones((2, 8), dtype=np.int32)
    with pytest.raises(B.MoeError):
        B.moe_ep_plan(np.ones((3, 8), dtype=np.int32), 0)          # E not divisible by R
    with pytest.raises(B.MoeError):
        B.moe_ep_plan(c, 2)                                        # rank out of range
    with pytest.raises(B.MoeError):
        B.moe_ep_plan(-c, 0)


_WORKER = r"""
import os, sys
import numpy as np
import torch, torch.distributed as dist
sys.path.insert(0, sys.argv[1])
from paper_2605_23764_b200 import binding as B
from oracle import ep_oracle
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:" + sys.argv[2], rank=int(sys.argv[3]), world_size=2)
rank, R, E, k, d = dist.get_rank(), 2, 8, 2, 4
Ts = [61, 90]
rng = np.random.default_rng(100 + rank)                           # each rank knows only its own tokens and routing
x = rng.normal(size=(Ts[rank], d))
ids = np.array([rng.permutation(E)[:k] for _ in range(Ts[rank])], dtype=np.int32)
w = rng.uniform(0.1, 1.0, size=(Ts[rank], k))
mine = torch.from_numpy(np.bincount(ids.reshape(-1), minlength=E).astype(np.int32))
gathered = [torch.empty_like(mine) for _ in range(R)]
dist.all_gather(gathered, mine)                                   # the metadata exchange that precedes Dispatch
counts = torch.stack(gathered).numpy()
tasks, recv_rows, offs = B.moe_ep_plan(counts, rank)
# "remote writes": every rank sends (destination, row, payload) for its tasks; the destination applies what it receives
src_of = np.argsort(ids.reshape(-1), kind="stable")
outgoing = [[] for _ in range(R)]
for e, r0, n, q, d0 in tasks:
    for r in range(n):
        slot = int(src_of[r0 + r])
        outgoing[q].append((int(d0 + r), rank, slot, x[slot // k].tolist(), float(w.reshape(-1)[slot])))
allout = [None] * R
dist.all_gather_object(allout, outgoing)
recv = np.full((recv_rows[rank], d), np.nan); meta = np.full((recv_rows[rank], 2), -1)
for s in range(R):
    for row, src, slot, payload, wt in allout[s][rank]:
        assert np.isnan(recv[row, 0])
        recv[row] = payload; meta[row] = (src, slot)
# every rank checks its receive buffer against the oracle run on the gathered problem
allx, allids, allw = [None] * R, [None] * R, [None] * R
dist.all_gather_object(allx, x); dist.all_gather_object(allids, ids); dist.all_gather_object(allw, w)
ref = ep_oracle.ep_dispatch(allx, allids, allw, E)[rank]
assert np.array_equal(recv, ref["rows"]) and np.array_equal(meta, ref["meta"]) and np.array_equal(offs, ref["expert_offsets"])
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_two_ranks_over_gloo_agree_with_the_oracle(tmp_path):
    script = tmp_path / "ep_worker.py"
    script.write_text(_WORKER)
    port = str(29500 + os.getpid() % 2000)
    procs = [subprocess.Popen([sys.executable, str(script), ROOT, port, str(r)], stdout=subprocess.PIPE, stderr=subprocess.STDOUT,
                              text=True) for r in range(2)]
    outs = [p.communicate(timeout=240)[0] for p in procs]
    for r, (p, o) in enumerate(zip(procs, outs)):
        assert p.returncode == 0 and f"rank {r} ok" in o, o
