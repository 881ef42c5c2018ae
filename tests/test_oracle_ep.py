"""Pins of the expert-parallel Dispatch / Combine oracle (Section 2.2, Section 4.1).  CPU only."""
import numpy as np

import oracle
from oracle import ep_oracle


def _problem(R, E, k, d, Ts, seed):
    rng = np.random.default_rng(seed)
    x = [rng.normal(size=(T, d)) for T in Ts]
    ids = [np.array([rng.permutation(E)[:k] for _ in range(T)], dtype=np.int32).reshape(T, k) for T in Ts]
    w = [rng.uniform(0.1, 1.0, size=(T, k)) for T in Ts]
    return x, ids, w


def test_dispatch_equals_the_single_device_layout_of_the_ranks_tokens_laid_end_to_end():
    R, E, k, d, Ts = 4, 8, 3, 5, [7, 0, 12, 5]
    x, ids, w = _problem(R, E, k, d, Ts, 1)
    got = ep_oracle.ep_dispatch(x, ids, w, E)
    # the pinned single-device layout on the concatenated tokens: expert-ordered rows, stable by global slot
    xg, idg = np.concatenate(x), np.concatenate(ids)
    counts, offsets, row_of, src_of = oracle.layout(idg, E)
    starts = np.cumsum([0] + Ts)
    El = E // R
    for q in range(R):
        lo, hi = offsets[q * El], offsets[(q + 1) * El]
        slots = src_of[lo:hi]                                   # global slots of the rows rank q must receive, in order
        np.testing.assert_array_equal(got[q]["rows"], xg[slots // k])
        src_rank = np.searchsorted(starts, slots // k, side="right") - 1
        np.testing.assert_array_equal(got[q]["meta"][:, 0], src_rank)
        np.testing.assert_array_equal(got[q]["meta"][:, 1], slots - starts[src_rank] * k)
        np.testing.assert_array_equal(got[q]["expert_offsets"], offsets[q * El:(q + 1) * El + 1] - lo)
        np.testing.assert_array_equal(got[q]["w"], np.concatenate(w).reshape(-1)[slots])


def test_dispatch_tiny_case_by_hand():
    # 2 ranks, 2 experts (expert 0 on rank 0, expert 1 on rank 1), k = 1
    x = [np.array([[1.0], [2.0]]), np.array([[3.0]])]
    ids = [np.array([[1], [0]], dtype=np.int32), np.array([[0]], dtype=np.int32)]
    w = [np.array([[0.5], [0.25]]), np.array([[1.0]])]
    got = ep_oracle.ep_dispatch(x, ids, w, 2)
    np.testing.assert_array_equal(got[0]["rows"], [[2.0], [3.0]])        # expert 0: rank 0's token 1, then rank 1's token 0
    np.testing.assert_array_equal(got[0]["meta"], [[0, 1], [1, 0]])
    np.testing.assert_array_equal(got[1]["rows"], [[1.0]])
    np.testing.assert_array_equal(got[1]["meta"], [[0, 0]])
    np.testing.assert_array_equal(got[0]["w"], [0.25, 1.0])


def test_arrival_counts_sum_to_the_rows_each_rank_receives():
    R, E, k, d, Ts = 2, 8, 2, 3, [100, 37]
    x, ids, w = _problem(R, E, k, d, Ts, 2)
    disp = ep_oracle.ep_dispatch(x, ids, w, E)
    thr = ep_oracle.ep_arrival_counts(ids, E, 32)
    for q in range(R):
        n = disp[q]["rows"].shape[0]
        assert thr[q].sum() == n and len(thr[q]) == -(-n // 32) and np.all(thr[q][:-1] == 32)
    assert sum(t.sum() for t in thr) == sum(Ts) * k


def test_dispatch_expert_combine_is_the_single_device_layer():
    R, E, k, d, F, Ts = 2, 4, 2, 8, 6, [9, 14]
    x, ids, w = _problem(R, E, k, d, Ts, 3)
    rng = np.random.default_rng(9)
    Wgu, Wd = rng.normal(size=(E, 2 * F, d)) / np.sqrt(d), rng.normal(size=(E, d, F)) / np.sqrt(F)
    disp = ep_oracle.ep_dispatch(x, ids, w, E)
    El = E // R
    y = []
    for q in range(R):                                           # each rank's experts on the rows it received (k = 1 there)
        offs = disp[q]["expert_offsets"]
        eid = np.repeat(np.arange(El), np.diff(offs)).astype(np.int32).reshape(-1, 1)
        y.append(oracle.fwd(disp[q]["rows"], eid, disp[q]["w"].reshape(-1, 1), Wgu[q * El:(q + 1) * El], Wd[q * El:(q + 1) * El]))
    out = ep_oracle.ep_combine(y, [dq["meta"] for dq in disp], Ts, k)
    ref = oracle.fwd(np.concatenate(x), np.concatenate(ids), np.concatenate(w), Wgu, Wd)
    np.testing.assert_allclose(np.concatenate(out), ref, rtol=1e-12, atol=1e-13)
