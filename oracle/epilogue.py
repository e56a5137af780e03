"""Statistics epilogue and Stage-2 rebalancing, written out plainly.  TEST INFRASTRUCTURE ONLY.

ochiai        Ochiai similarity of expert pairs (footnote of Section 1): |A n B| / sqrt(|A| |B|) for the
              token sets A, B of two experts, i.e. c_ij / sqrt(c_ii c_jj) on the co-activation counts.
ema_update    exponential moving average of a per-step count (Section 3.2: w^_e, c^_ij, w_er are EMAs;
              the paper gives no decay constant, so it is a parameter): ema <- decay*ema + (1-decay)*count.
rebalance_intra_node
              Stage 2 of the layout planner (Section 3.2): per node, the replicas are re-partitioned among
              the node's ranks by greedy bin packing on their EMA loads.  Reading taken: replicas sorted by
              load descending (ties: lower expert id, then lower old slot); each goes to the rank of its
              node with the smallest accumulated load among the ranks that still have a free slot (at most
              S replicas per rank, the (1+rho)E/G budget) and do not hold that expert yet (ties: lower
              rank); a rank's slots are filled in placement order.  If some replica finds no admissible
              rank, that node keeps its old placement.
"""
from __future__ import annotations

import numpy as np


def ochiai(coact: np.ndarray) -> np.ndarray:
    c = np.asarray(coact, dtype=np.float64)
    d = np.diag(c)
    denom = np.sqrt(np.outer(d, d))
    out = np.zeros_like(c)
    nz = denom > 0
    out[nz] = c[nz] / denom[nz]
    return out


def ema_update(ema: np.ndarray, counts: np.ndarray, decay: float) -> np.ndarray:
    return decay * np.asarray(ema, dtype=np.float64) + (1.0 - decay) * np.asarray(counts, dtype=np.float64)


def rebalance_intra_node(N: int, Q: int, S: int, slot_expert, load):
    """-> (new_slot_expert int32 [G*S], moved_from int32 [G*S] (old slot of each new slot, -1 if empty),
           nodes_kept: list of nodes whose placement could not be improved upon by the greedy pass)."""
    slot_expert = np.asarray(slot_expert, dtype=np.int64)
    load = np.asarray(load, dtype=np.float64)
    G = N * Q
    new = np.full(G * S, -1, dtype=np.int32)
    moved = np.full(G * S, -1, dtype=np.int32)
    kept = []
    for n in range(N):
        lo, hi = n * Q * S, (n + 1) * Q * S
        replicas = [(d, int(slot_expert[d]), float(load[d])) for d in range(lo, hi) if slot_expert[d] >= 0]
        replicas.sort(key=lambda r: (-r[2], r[1], r[0]))
        rank_load = [0.0] * Q
        rank_has = [[] for _ in range(Q)]
        placed = []                                    # (rank, position, old slot, expert)
        ok = True
        for d, e, w in replicas:
            best = None
            for q in range(Q):
                if len(rank_has[q]) >= S or e in rank_has[q]:
                    continue
                if best is None or rank_load[q] < rank_load[best]:
                    best = q
            if best is None:
                ok = False
                break
            placed.append((best, len(rank_has[best]), d, e))
            rank_has[best].append(e)
            rank_load[best] += w
        if not ok:
            kept.append(n)
            new[lo:hi] = slot_expert[lo:hi]
            for d in range(lo, hi):
                moved[d] = d if slot_expert[d] >= 0 else -1
            continue
        for q, pos, d, e in placed:
            slot = (n * Q + q) * S + pos
            new[slot] = e
            moved[slot] = d
    return new, moved, kept
