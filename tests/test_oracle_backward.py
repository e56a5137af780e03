"""Pins for the oracle's backward of the row stages (CPU only): adjoint identities against the
already-pinned forward oracle, and derivative-by-difference for the gate weights (the forward
map is linear in each argument, so unit differences are exact up to rounding)."""
import numpy as np

import oracle as O
import workloads as W


def _setup(T=150, H=48, name="3"):
    w = W.make_config(name, T=T)
    r = O.assign(w.N, w.Q, w.S, w.E, w.slot_expert, w.primary_slot, w.topk_ids, w.src_rank, w.seed)
    x = w.hidden_rows()[:, :H].copy()
    p = O.permute(r["assigned_slot"], w.D, x)
    out = w.expert_out_rows()[:, :H].copy()
    rng = np.random.default_rng(3)
    gy = W.bf16_bits_from_f32(rng.standard_normal((w.T, H)).astype(np.float32))
    gs = W.bf16_bits_from_f32(rng.standard_normal((w.P, H)).astype(np.float32))
    return w, p, x, out, gy, gs


def test_permute_backward_is_the_adjoint_of_the_gather():
    """<send(x), g> = <x, grad_x(g)> for the dispatch gather send[row(t,k)] = x[t]."""
    w, p, x, out, gy, gs = _setup()
    send = W.f32_from_bf16_bits(p["send"]).astype(np.float64)
    g = W.f32_from_bf16_bits(gs).astype(np.float64)
    grad_x = O.permute_backward(gs, p["row_of_pair"], w.T, w.K)
    lhs = (send * g).sum()
    rhs = (W.f32_from_bf16_bits(x).astype(np.float64) * grad_x).sum()
    assert abs(lhs - rhs) <= 1e-9 * max(1.0, abs(lhs))
    # token by token it is the plain sum of the token's K rows
    rows = p["row_of_pair"].reshape(w.T, w.K)
    assert np.allclose(grad_x, g[rows].sum(axis=1), rtol=0, atol=1e-12)


def test_combine_backward_is_the_adjoint_of_the_forward_oracle():
    """<y(out), u> = <out, grad_out(u)>, with y from the (separately pinned) forward oracle."""
    w, p, x, out, gy, gs = _setup()
    y = O.combine(out, p["row_of_pair"], w.gate_w).astype(np.float64)
    u = W.f32_from_bf16_bits(gy).astype(np.float64)
    grad_out, grad_w = O.combine_backward(gy, out, p["row_of_pair"], w.gate_w)
    lhs = (y * u).sum()
    rhs = (W.f32_from_bf16_bits(out).astype(np.float64) * grad_out).sum()
    scale = (np.abs(y) * np.abs(u)).sum()
    assert abs(lhs - rhs) <= 1e-6 * scale        # y carries fp32 rounding


def test_gate_weight_gradient_by_unit_difference():
    """y is linear in g: <y(g + e_tk) - y(g), u> = grad_g[t][k]."""
    w, p, x, out, gy, gs = _setup(T=40, H=32)
    u = W.f32_from_bf16_bits(gy).astype(np.float64)
    _, grad_w = O.combine_backward(gy, out, p["row_of_pair"], w.gate_w)
    zero = np.zeros_like(w.gate_w)
    for t, k in [(0, 0), (7, 3), (39, 5), (20, 1)]:
        e = zero.copy()
        e[t, k] = 1.0
        dy = O.combine(out, p["row_of_pair"], e).astype(np.float64)      # forward of the unit weight alone
        fd = (dy * u).sum()
        assert abs(fd - grad_w[t, k]) <= 1e-9 * max(1.0, np.abs(u[t]).sum() * 10)


def test_backward_special_cases():
    w, p, x, out, gy, gs = _setup(T=60, H=16)
    grad_out, grad_w = O.combine_backward(gy, out, p["row_of_pair"], np.ones_like(w.gate_w))
    u = W.f32_from_bf16_bits(gy).astype(np.float64)
    rows = p["row_of_pair"].reshape(w.T, w.K)
    for k in range(w.K):
        assert (grad_out[rows[:, k]] == u).all()          # unit weights copy grad_y to every row
    grad_out0, _ = O.combine_backward(gy, out, p["row_of_pair"], np.zeros_like(w.gate_w))
    assert (grad_out0 == 0).all()
    # identity experts (out = send): grad_g[t][k] = <grad_y[t], x[t]> for every k
    _, gw = O.combine_backward(gy, p["send"], p["row_of_pair"], w.gate_w)
    dots = (u * W.f32_from_bf16_bits(x).astype(np.float64)).sum(axis=1)
    assert np.allclose(gw, dots[:, None], rtol=1e-12, atol=1e-12)
