"""Oracle of expert-parallel Dispatch / Combine (Section 2.2: Dispatch sends every routed token copy to the rank that
hosts its expert, Combine returns the expert outputs to the token's rank and accumulates the top-k contributions;
Section 4.1: both are sets of independent remote writes, each with a completion counter on the destination).

TEST INFRASTRUCTURE ONLY: plain Python / numpy loops in definition order, no code shared with the CUDA path.

R ranks; rank s holds tokens x[s] [T_s, d] with ids[s] [T_s, k] (global expert ids) and w[s] [T_s, k]; expert e lives on
rank e // (E / R).  On the destination the rows of one expert are ordered by source rank, then by the source's flat slot
index t*k + j (the single-device rule -- stable by slot -- applied to the ranks' tokens laid end to end).
"""
from __future__ import annotations

import numpy as np


def ep_dispatch(x, ids, w, E):
    """-> per destination rank q: rows [n_q, d] (float64 copy of the source rows), meta int64 [n_q, 2] = (source rank,
    source slot), weight float64 [n_q], expert_offsets int64 [E/R + 1] (first row of each local expert)."""
    R = len(x)
    assert E % R == 0
    El = E // R
    out = []
    for q in range(R):
        rows, meta, wt, offs = [], [], [], [0]
        for e in range(q * El, (q + 1) * El):
            for s in range(R):
                T, k = ids[s].shape
                for t in range(T):
                    for j in range(k):
                        if ids[s][t, j] == e:
                            rows.append(np.asarray(x[s][t], dtype=np.float64))
                            meta.append((s, t * k + j))
                            wt.append(float(w[s][t, j]))
            offs.append(len(rows))
        d = np.asarray(x[0]).shape[1]
        out.append({"rows": np.array(rows, dtype=np.float64).reshape(len(rows), d),
                    "meta": np.array(meta, dtype=np.int64).reshape(len(meta), 2),
                    "w": np.array(wt, dtype=np.float64), "expert_offsets": np.array(offs, dtype=np.int64)})
    return out


def ep_arrival_counts(ids, E, block_rows):
    """Rows that land in each block of `block_rows` rows of every destination's receive buffer: the thresholds its
    completion counters must reach.  -> list over ranks of int64 arrays."""
    R = len(ids)
    El = E // R
    out = []
    for q in range(R):
        n = sum(int(np.sum((ids[s] >= q * El) & (ids[s] < (q + 1) * El))) for s in range(R))
        nb = -(-n // block_rows)
        out.append(np.array([min(block_rows, n - b * block_rows) for b in range(nb)], dtype=np.int64))
    return out


def ep_combine(y_rows, meta, T_list, k):
    """Return every expert-output row to (source rank, slot) and sum each token's k rows in slot order.
    y_rows[q] [n_q, d], meta[q] [n_q, 2] -> out[s] float64 [T_s, d]."""
    R = len(T_list)
    d = y_rows[0].shape[1]
    ret = [np.zeros((T_list[s] * k, d)) for s in range(R)]
    seen = [np.zeros(T_list[s] * k, dtype=np.int64) for s in range(R)]
    for q in range(R):
        for p in range(y_rows[q].shape[0]):
            s, slot = int(meta[q][p, 0]), int(meta[q][p, 1])
            ret[s][slot] = y_rows[q][p]
            seen[s][slot] += 1
    for s in range(R):
        assert np.all(seen[s] == 1), "every slot returns exactly once"
    return [ret[s].reshape(T_list[s], k, d).sum(axis=1) for s in range(R)]
