"""GPU parity of the node-deduplicated send layout against the oracle (bit-exact)."""
import numpy as np
import pytest
import torch

import oracle as O
import workloads as W
from gpu_util import bits_from_bf16_tensor, make_step, oracle_assign, u32

pytestmark = pytest.mark.gpu


def _dedup_buffers(w):
    dev = "cuda"
    return dict(node_counts=torch.zeros(w.N, dtype=torch.int32, device=dev),
                node_offsets=torch.zeros(w.N + 1, dtype=torch.int32, device=dev),
                node_row=torch.zeros(w.T * w.N, dtype=torch.int32, device=dev),
                fwd=torch.zeros(w.P, dtype=torch.int32, device=dev),
                cross=torch.zeros(1, dtype=torch.int64, device=dev))


@pytest.mark.parametrize("name,T", [("1", 4096), ("1a", 4096), ("2", 5000), ("3", 7001), ("5", 3000)])
def test_dedup_layout_elementwise(name, T):
    import paper_2609_36959_b200 as cb
    w = W.make_config(name, T=T)
    layout, step = make_step(w, alias_expert_out=False)
    step.route(w.seed)
    b = _dedup_buffers(w)
    ws = torch.empty(cb.dedup_workspace_bytes(w.T, w.K, w.N), dtype=torch.uint8, device="cuda")
    for _ in range(2):
        cb.dedup_index(step.assigned_slot, step.src_rank, w.N, w.Q, w.S, b["node_counts"], b["node_offsets"],
                       b["node_row"], b["fwd"], ws, cross_node_rows=b["cross"])
    torch.cuda.synchronize()
    r = oracle_assign(w, w.seed)
    d = O.dedup_index(r["assigned_slot"], w.src_rank, w.N, w.Q, w.S)
    assert (u32(b["node_counts"]) == d["node_counts"]).all()
    assert (u32(b["node_offsets"]) == d["node_offsets"]).all()
    assert (b["node_row"].cpu().numpy().reshape(w.T, w.N) == d["node_row_of_token"]).all()
    assert (b["fwd"].cpu().numpy() == d["fwd_src_row"]).all()
    assert int(b["cross"][0]) == d["cross_node_rows"] == int(step.totals[0])

    total = int(d["node_offsets"][-1])
    dedup_send = torch.zeros((total, w.H), dtype=torch.bfloat16, device="cuda")
    cb.dedup_rows(step.x, b["node_row"], w.N, dedup_send)
    recv = torch.zeros_like(step.send)
    cb.forward_rows(dedup_send, b["fwd"], step.row_of_pair, recv)
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0
    x = w.hidden_rows()
    assert (bits_from_bf16_tensor(dedup_send) == O.dedup_rows(x, d["node_row_of_token"], total)).all()
    assert torch.equal(recv.view(torch.int16), step.send.view(torch.int16))      # same buffer as cobalt_permute


def test_dedup_full_size_config5():
    import paper_2609_36959_b200 as cb
    w = W.make_config("5")
    layout, step = make_step(w, alias_expert_out=True)
    step.route(w.seed)
    b = _dedup_buffers(w)
    ws = torch.empty(cb.dedup_workspace_bytes(w.T, w.K, w.N), dtype=torch.uint8, device="cuda")
    cb.dedup_index(step.assigned_slot, step.src_rank, w.N, w.Q, w.S, b["node_counts"], b["node_offsets"],
                   b["node_row"], b["fwd"], ws, cross_node_rows=b["cross"])
    torch.cuda.synchronize()
    r = oracle_assign(w, w.seed)
    d = O.dedup_index(r["assigned_slot"], w.src_rank, w.N, w.Q, w.S)
    assert (u32(b["node_offsets"]) == d["node_offsets"]).all()
    assert (b["node_row"].cpu().numpy().reshape(w.T, w.N) == d["node_row_of_token"]).all()
    assert (b["fwd"].cpu().numpy() == d["fwd_src_row"]).all()
    assert int(b["cross"][0]) == r["V"]
    total = int(d["node_offsets"][-1])
    assert total < w.P
    dedup_send = torch.zeros((total, w.H), dtype=torch.bfloat16, device="cuda")
    cb.dedup_rows(step.x, b["node_row"], w.N, dedup_send)
    ref = step.send.clone()
    step.send.zero_()
    cb.forward_rows(dedup_send, b["fwd"], step.row_of_pair, step.send)
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0
    assert torch.equal(step.send.view(torch.int16), ref.view(torch.int16))
