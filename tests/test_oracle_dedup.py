"""Pins for the oracle's node-deduplicated send layout (CPU only)."""
import numpy as np
import pytest

import oracle as O
import workloads as W


@pytest.mark.parametrize("name,T", [("1", 1500), ("2", 1000), ("3", 1200), ("5", 600)])
def test_dedup_layout_reproduces_the_plain_send_buffer(name, T):
    w = W.make_config(name, T=T)
    r = O.assign(w.N, w.Q, w.S, w.E, w.slot_expert, w.primary_slot, w.topk_ids, w.src_rank, w.seed)
    x = w.hidden_rows()[:, :32].copy()
    p = O.permute(r["assigned_slot"], w.D, x)
    d = O.dedup_index(r["assigned_slot"], w.src_rank, w.N, w.Q, w.S)
    total = int(d["node_offsets"][-1])
    buf = O.dedup_rows(x, d["node_row_of_token"], total)
    # forwarding on the receiving node rebuilds exactly the destination-grouped buffer
    assert (O.forward_rows(buf, d["fwd_src_row"], p["row_of_pair"]) == p["send"]).all()
    # the number of rows that cross a node boundary is Eq. 1's V
    V, _ = O.traffic(w.N, w.Q, w.S, w.E, w.slot_expert, w.topk_ids, w.src_rank, r["assigned_slot"])
    assert d["cross_node_rows"] == V == r["V"]
    # one row per distinct (token, node): counted independently with numpy
    spn = w.S * w.Q
    pairs = np.unique(np.stack([np.repeat(np.arange(w.T), w.K), (r["assigned_slot"] // spn).ravel()], 1), axis=0)
    assert total == len(pairs) <= w.P
    assert (d["node_counts"] == np.bincount(pairs[:, 1], minlength=w.N)).all()
    # rows of one node are in ascending token order and hold that token's row
    for n in range(w.N):
        rows = d["node_row_of_token"][:, n]
        toks = np.nonzero(rows >= 0)[0]
        assert (rows[toks] == d["node_offsets"][n] + np.arange(len(toks))).all()
        assert (buf[rows[toks]] == x[toks]).all()
    if name != "2":
        assert total < w.P                  # some token reaches two experts on one node


def test_dedup_tiny_by_hand():
    # 2 nodes x 1 rank x 2 slots; tokens: t0 -> slots 0,1 (node 0 twice); t1 -> slots 1,2 (nodes 0,1); t2 -> 3,2 (node 1 twice)
    slots = np.array([[0, 1], [1, 2], [3, 2]], np.int32)
    d = O.dedup_index(slots, np.array([0, 0, 1], np.int32), 2, 1, 2)
    assert d["node_counts"].tolist() == [2, 2] and d["node_offsets"].tolist() == [0, 2, 4]
    assert d["node_row_of_token"].tolist() == [[0, -1], [1, 2], [-1, 3]]
    assert d["fwd_src_row"].tolist() == [0, 0, 1, 2, 3, 3]
    assert d["cross_node_rows"] == 1          # only t1 leaves its node (source node 0 -> node 1)
