"""Node-deduplicated send layout, written out plainly.  TEST INFRASTRUCTURE ONLY.

Section 3.1 (and Section 1 on DeepEP): when several ranks of one node need the same token, it
crosses the network once and is forwarded inside the node, which is why Eq. 1 counts distinct
destination nodes.  The buffer that realises this holds ONE row per (token, destination node),
grouped by destination node in ascending token order, plus, for every (token, expert) pair, the
row of that buffer it is forwarded from on the receiving node.
"""
from __future__ import annotations

import numpy as np


def dedup_index(assigned_slot: np.ndarray, src_rank: np.ndarray, N: int, Q: int, S: int):
    """-> dict(node_counts [N], node_offsets [N+1], node_row_of_token [T,N] (-1 where the token does not
    go to that node), fwd_src_row [T*K], cross_node_rows = Eq. 1's V)."""
    slots = np.asarray(assigned_slot, dtype=np.int64)
    T, K = slots.shape
    spn = S * Q
    node_of_pair = slots // spn
    lists = [[] for _ in range(N)]
    for t in range(T):
        for n in sorted(set(node_of_pair[t].tolist())):
            lists[n].append(t)
    counts = np.array([len(l) for l in lists], dtype=np.uint32)
    offsets = np.zeros(N + 1, dtype=np.uint32)
    offsets[1:] = np.cumsum(counts)
    node_row = np.full((T, N), -1, dtype=np.int32)
    for n in range(N):
        for i, t in enumerate(lists[n]):
            node_row[t, n] = offsets[n] + i
    fwd = node_row[np.arange(T)[:, None], node_of_pair].astype(np.int32).reshape(-1)
    src_node = np.asarray(src_rank, dtype=np.int64) // Q
    cross = int(sum(len(set(node_of_pair[t].tolist()) - {int(src_node[t])}) for t in range(T)))
    return dict(node_counts=counts, node_offsets=offsets, node_row_of_token=node_row, fwd_src_row=fwd,
                cross_node_rows=cross)


def dedup_rows(x_bits: np.ndarray, node_row_of_token: np.ndarray, total_rows: int) -> np.ndarray:
    out = np.zeros((total_rows, x_bits.shape[1]), dtype=np.uint16)
    T, N = node_row_of_token.shape
    for t in range(T):
        for n in range(N):
            r = node_row_of_token[t, n]
            if r >= 0:
                out[r] = x_bits[t]
    return out


def forward_rows(dedup_send: np.ndarray, fwd_src_row: np.ndarray, row_of_pair: np.ndarray) -> np.ndarray:
    """The receiving node's expansion: recv[row_of_pair[p]] = dedup_send[fwd_src_row[p]]."""
    recv = np.zeros((len(row_of_pair), dedup_send.shape[1]), dtype=np.uint16)
    for p in range(len(row_of_pair)):
        recv[row_of_pair[p]] = dedup_send[fwd_src_row[p]]
    return recv
