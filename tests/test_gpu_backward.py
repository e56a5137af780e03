"""GPU parity of the backward of the row stages against the oracle's adjoints (float64).

Tolerances: bf16 outputs as for the combine, |gpu - ref| <= 1e-2 + 1e-2 |ref|; the fp32 gate-weight
gradient within 1e-4 of the sum of the absolute terms of its dot product (the bound of an fp32
summation of H terms in any order is H * 2^-24 of that sum; H <= 16384 here)."""
import numpy as np
import pytest
import torch

import oracle as O
import workloads as W
from gpu_util import bf16_tensor_from_bits, bits_from_bf16_tensor, make_step, oracle_assign

pytestmark = pytest.mark.gpu


def _close_bf16(got_bits, ref):
    got = W.f32_from_bf16_bits(got_bits).astype(np.float64)
    err = np.abs(got - ref)
    assert (err <= 1e-2 + 1e-2 * np.abs(ref)).all(), float(err.max())


def _random_bf16(shape, seed):
    rng = np.random.default_rng(seed)
    return W.bf16_bits_from_f32(rng.standard_normal(shape, dtype=np.float32))


@pytest.mark.parametrize("name,T,H", [("1", 4096, 1024), ("2", 3000, 4096), ("3", 5000, 2048), ("5", 700, 7168)])
def test_backward_elementwise(name, T, H):
    import paper_2609_36959_b200 as cb
    w = W.make_config(name, T=T)
    assert w.H == H
    layout, step = make_step(w, alias_expert_out=False)
    r = oracle_assign(w, w.seed)
    p = O.permute(r["assigned_slot"], w.D)
    step.assign(w.seed)
    cb.permute_index(step.assigned_slot, w.D, step.dest_counts, step.dest_offsets, step.row_of_pair,
                     step.pair_of_row, step.workspace)
    out = w.expert_out_rows()
    gy = _random_bf16((w.T, w.H), 11)
    gs = _random_bf16((w.P, w.H), 12)
    step.expert_out.copy_(bf16_tensor_from_bits(out, "cpu"))
    gy_d = bf16_tensor_from_bits(gy)
    gs_d = bf16_tensor_from_bits(gs)
    grad_x = torch.zeros_like(step.x)
    grad_out = torch.zeros_like(step.send)
    grad_w = torch.zeros_like(step.gate_w)

    cb.permute_backward(gs_d, step.row_of_pair, w.K, grad_x)
    cb.combine_backward(gy_d, step.expert_out, step.row_of_pair, step.gate_w, grad_out, grad_w)
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0

    _close_bf16(bits_from_bf16_tensor(grad_x), O.permute_backward(gs, p["row_of_pair"], w.T, w.K))
    ref_out, ref_w = O.combine_backward(gy, out, p["row_of_pair"], w.gate_w)
    _close_bf16(bits_from_bf16_tensor(grad_out), ref_out)
    rows = p["row_of_pair"].reshape(w.T, w.K)
    terms = np.abs(W.f32_from_bf16_bits(gy).astype(np.float64)[:, None, :] *
                   W.f32_from_bf16_bits(out).astype(np.float64)[rows]).sum(axis=2)
    assert (np.abs(grad_w.cpu().numpy().astype(np.float64) - ref_w) <= 1e-4 * terms + 1e-30).all()

    # either output alone, and run-to-run identical bits
    grad_out2 = torch.zeros_like(grad_out)
    grad_w2 = torch.zeros_like(grad_w)
    cb.combine_backward(gy_d, None, step.row_of_pair, step.gate_w, grad_out2, None)
    cb.combine_backward(gy_d, step.expert_out, step.row_of_pair, step.gate_w, None, grad_w2)
    torch.cuda.synchronize()
    assert torch.equal(grad_out2.view(torch.int16), grad_out.view(torch.int16))
    assert torch.equal(grad_w2, grad_w)


def test_backward_full_size_properties():
    """Config 5 at full size: exact closed forms that hold for any size, plus sampled oracle rows."""
    import paper_2609_36959_b200 as cb
    w = W.make_config("5")
    layout, step = make_step(w, alias_expert_out=True)
    step.route(w.seed)                                   # send = rows of x (identity experts)
    grad_x = torch.zeros_like(step.x)
    cb.permute_backward(step.send, step.row_of_pair, w.K, grad_x)
    torch.cuda.synchronize()
    # the K rows of a token all hold x[t]: their sum is K * x[t], exact in bf16 for K = 8
    # (compared as values: the sum of zeros is +0 whatever their signs)
    assert bool((grad_x.float() == step.x.float() * w.K).all())

    gy = step.y                                          # any bf16 [T, H] tensor serves as grad_y
    grad_w = torch.zeros_like(step.gate_w)
    grad_out = torch.empty_like(step.send)
    cb.combine_backward(gy, step.send, step.row_of_pair, step.gate_w, grad_out, grad_w)
    torch.cuda.synchronize()
    assert cb.read_and_clear_device_error() == 0
    rng = np.random.default_rng(9)
    tokens = np.unique(np.concatenate([rng.integers(0, w.T, 300), [0, w.T - 1]]))
    tok = torch.from_numpy(tokens).cuda()
    rows = step.row_of_pair.view(w.T, w.K)[tok].cpu().numpy()            # [n, K]
    gy_bits = bits_from_bf16_tensor(gy[tok])
    out_bits = bits_from_bf16_tensor(step.send[torch.from_numpy(rows.ravel()).cuda()])
    ref_out, ref_w = O.combine_backward(gy_bits, out_bits, np.arange(rows.size, dtype=np.int32), w.gate_w[tokens])
    got_out = bits_from_bf16_tensor(grad_out[torch.from_numpy(rows.ravel()).cuda()])
    _close_bf16(got_out, ref_out)
    terms = np.abs(W.f32_from_bf16_bits(gy_bits).astype(np.float64)[:, None, :] *
                   W.f32_from_bf16_bits(out_bits).astype(np.float64).reshape(len(tokens), w.K, w.H)).sum(axis=2)
    got_w = grad_w[tok].cpu().numpy().astype(np.float64)
    assert (np.abs(got_w - ref_w) <= 1e-4 * terms + 1e-30).all()
    # identity experts: every k of a token sees the same row, so the K gate gradients are equal
    assert bool((grad_w == grad_w[:, :1]).all())
