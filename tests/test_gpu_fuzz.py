"""Seeded random shapes through every stage (separate calls, fused pass, round-robin pick, dedup
layout, backward), each compared with the oracle.  Shapes are drawn from the supported envelope
with odd sizes on purpose: non-power-of-two E and D, K from 1 to 16, 1 to 8 nodes, empty slots,
ragged T."""
import os

import numpy as np
import pytest
import torch

import oracle as O
import workloads as W
from gpu_util import assert_combine_close, bf16_tensor_from_bits, bits_from_bf16_tensor, make_step, u32

pytestmark = pytest.mark.gpu


# COBALT_FUZZ_CASES=n runs n cases instead of 24; cases from 24 on draw from a wider envelope
N_CASES = int(os.environ.get("COBALT_FUZZ_CASES", "24"))


def _draw_shape(rng, wide=False):
    N = int(rng.choice([1, 2, 3, 4, 5, 8]))
    Q = int(rng.integers(1, 5))
    G = N * Q
    K = int(rng.choice([1, 2, 3, 4, 5, 6, 7, 8, 12, 16]))
    E = int(rng.integers(max(K, 2), 1025 if wide else 200))
    per = -(-E // G)
    S = per + int(rng.integers(0, 3))
    if E < G:
        S = 1
    while G * S > 4096:
        S -= 1
    T = int(rng.choice([1, 2, 31, 32, 33, 255, 256, 257, 1000, 2047, 2049, 5000, 9999] + ([20000, 40001] if wide else [])))
    H = 8 * int(rng.integers(1, 40))
    empty = int(rng.integers(0, 3)) if E >= G else 0
    return T, E, K, H, N, Q, S, empty


@pytest.mark.parametrize("case", range(N_CASES))
def test_random_shape(case):
    import paper_2609_36959_b200 as cb
    rng = np.random.default_rng(1000 + case)
    T, E, K, H, N, Q, S, empty = _draw_shape(rng, wide=case >= 24)
    w = W.make_custom(T, E, K, H, N, Q, S, seed=500 + case, C=int(rng.integers(1, 6)), p_in=0.6, n_empty=empty)
    seed = int(rng.integers(0, 2**63))
    layout, step = make_step(w, alias_expert_out=False)
    note = f"T={T} E={E} K={K} H={H} N={N} Q={Q} S={S} empty={empty}"

    coact, load = O.coact_stats(w.topk_ids, w.E)
    r = O.assign(w.N, w.Q, w.S, w.E, w.slot_expert, w.primary_slot, w.topk_ids, w.src_rank, seed)
    x = w.hidden_rows()
    p = O.permute(r["assigned_slot"], w.D, x)
    out = w.expert_out_rows()
    y_ref = O.combine(out, p["row_of_pair"], w.gate_w)

    def check_index():
        assert (u32(step.coact) == coact).all() and (u32(step.load) == load).all(), note
        assert (step.assigned_slot.cpu().numpy() == r["assigned_slot"]).all(), note
        assert (step.remote_nodes.cpu().numpy() == r["remote_nodes"]).all(), note
        assert step.totals.cpu().tolist() == [r["V"], r["V_naive"]], note
        assert (u32(step.dest_counts) == p["dest_counts"]).all(), note
        assert (u32(step.dest_offsets) == p["dest_offsets"]).all(), note
        assert (step.row_of_pair.cpu().numpy() == p["row_of_pair"]).all(), note
        assert (step.pair_of_row.cpu().numpy() == p["pair_of_row"]).all(), note

    # separate calls
    step.stats()
    step.assign(seed)
    step.permute()
    step.expert_out.copy_(bf16_tensor_from_bits(out, "cpu"))
    step.combine()
    torch.cuda.synchronize()
    check_index()
    assert (u32(step.slot_load) == r["slot_load"]).all(), note
    assert (bits_from_bf16_tensor(step.send) == p["send"]).all(), note
    assert_combine_close(bits_from_bf16_tensor(step.y), y_ref)

    # fused pass over used buffers
    for buf in (step.coact, step.assigned_slot, step.row_of_pair, step.dest_offsets, step.totals):
        buf.fill_(3)
    cb.route_index(layout, step.topk_ids, step.src_rank, seed, step.coact, step.load, step.assigned_slot,
                   step.dest_counts, step.dest_offsets, step.row_of_pair, step.workspace,
                   remote_nodes=step.remote_nodes, totals=step.totals, pair_of_row=step.pair_of_row)
    torch.cuda.synchronize()
    check_index()

    # round-robin pick
    if w.E * w.N <= 4096:
        rr = O.assign(w.N, w.Q, w.S, w.E, w.slot_expert, w.primary_slot, w.topk_ids, w.src_rank, seed,
                      round_robin=True)
        slots = torch.zeros_like(step.assigned_slot)
        cb.assign(layout, step.topk_ids, step.src_rank, seed, slots, slot_load=step.slot_load,
                  flags=cb.ASSIGN_ROUND_ROBIN, workspace=step.workspace)
        torch.cuda.synchronize()
        assert (slots.cpu().numpy() == rr["assigned_slot"]).all(), note
        assert (u32(step.slot_load) == rr["slot_load"]).all(), note

    # dedup layout and its expansion
    d = O.dedup_index(r["assigned_slot"], w.src_rank, w.N, w.Q, w.S)
    nc = torch.zeros(w.N, dtype=torch.int32, device="cuda")
    no = torch.zeros(w.N + 1, dtype=torch.int32, device="cuda")
    nr = torch.zeros(w.T * w.N, dtype=torch.int32, device="cuda")
    fwd = torch.zeros(w.P, dtype=torch.int32, device="cuda")
    cross = torch.zeros(1, dtype=torch.int64, device="cuda")
    ws = torch.empty(max(cb.dedup_workspace_bytes(w.T, w.K, w.N), 256), dtype=torch.uint8, device="cuda")
    cb.dedup_index(step.assigned_slot, step.src_rank, w.N, w.Q, w.S, nc, no, nr, fwd, ws, cross_node_rows=cross)
    torch.cuda.synchronize()
    assert (u32(no) == d["node_offsets"]).all() and (fwd.cpu().numpy() == d["fwd_src_row"]).all(), note
    assert int(cross[0]) == d["cross_node_rows"] == r["V"], note
    total = int(d["node_offsets"][-1])
    buf = torch.zeros((max(total, 1), w.H), dtype=torch.bfloat16, device="cuda")
    cb.dedup_rows(step.x, nr, w.N, buf)
    recv = torch.zeros_like(step.send)
    cb.forward_rows(buf, fwd, step.row_of_pair, recv)
    torch.cuda.synchronize()
    assert (bits_from_bf16_tensor(recv) == p["send"]).all(), note

    # backward
    gy = W.bf16_bits_from_f32(rng.standard_normal((w.T, w.H), dtype=np.float32))
    gs = W.bf16_bits_from_f32(rng.standard_normal((w.P, w.H), dtype=np.float32))
    grad_x = torch.zeros_like(step.x)
    grad_out = torch.zeros_like(step.send)
    grad_w = torch.zeros_like(step.gate_w)
    cb.permute_backward(bf16_tensor_from_bits(gs), step.row_of_pair, w.K, grad_x)
    cb.combine_backward(bf16_tensor_from_bits(gy), step.expert_out, step.row_of_pair, step.gate_w, grad_out, grad_w)
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0, note

    def close(bits, ref):
        got = W.f32_from_bf16_bits(bits).astype(np.float64)
        assert (np.abs(got - ref) <= 1e-2 + 1e-2 * np.abs(ref)).all(), note
    close(bits_from_bf16_tensor(grad_x), O.permute_backward(gs, p["row_of_pair"], w.T, w.K))
    ref_out, ref_w = O.combine_backward(gy, out, p["row_of_pair"], w.gate_w)
    close(bits_from_bf16_tensor(grad_out), ref_out)
    rows = p["row_of_pair"].reshape(w.T, w.K)
    terms = np.abs(W.f32_from_bf16_bits(gy).astype(np.float64)[:, None, :] *
                   W.f32_from_bf16_bits(out).astype(np.float64)[rows]).sum(axis=2)
    assert (np.abs(grad_w.cpu().numpy().astype(np.float64) - ref_w) <= 1e-4 * terms + 1e-30).all(), note
