"""Pins for the oracle's statistics, permutation and combine (CPU only)."""
import numpy as np
import pytest

import oracle as O
import workloads as W


# ---------------------------------------------------------------- statistics --------------
def test_stats_fig1_tokens(fig1):
    ids = np.array([tk["ids"] for tk in fig1["tokens"]], np.int32)
    coact, load = O.coact_stats(ids, 4)
    assert load.tolist() == fig1["load"]
    off = coact[~np.eye(4, dtype=bool)]
    assert (off == fig1["coact_offdiag"]).all()
    ochiai = coact / np.sqrt(np.outer(load, load))
    assert np.allclose(ochiai[~np.eye(4, dtype=bool)], fig1["ochiai_offdiag"])


@pytest.mark.parametrize("name,T", [("1", 4096), ("3", 5000), ("5", 3000)])
def test_stats_equal_indicator_gram_matrix(name, T):
    """coact = M^T M for the T x E 0/1 selection matrix (numpy), load = column sums."""
    w = W.make_config(name, T=T)
    coact, load = O.coact_stats(w.topk_ids, w.E)
    M = np.zeros((w.T, w.E), np.int64)
    M[np.arange(w.T)[:, None], w.topk_ids] = 1
    assert (coact == M.T @ M).all()
    assert (load == M.sum(axis=0)).all()


def test_stats_invariants():
    w = W.make_config("4", T=4000)
    coact, load = O.coact_stats(w.topk_ids, w.E)
    c = coact.astype(np.int64)
    assert (c == c.T).all()
    assert (np.diag(c) == load).all()
    assert (c.sum(axis=1) == w.K * load.astype(np.int64)).all()
    assert load.sum() == w.K * w.T and c.sum() == w.K * w.K * w.T
    # Ochiai similarity |A & B| / sqrt(|A||B|) lies in [0, 1]
    nz = load > 0
    och = c[np.ix_(nz, nz)] / np.sqrt(np.outer(load[nz], load[nz]))
    assert och.min() >= 0 and och.max() <= 1 + 1e-12


def test_stats_always_coselected_pair_has_ochiai_one():
    ids = np.array([[0, 1, 2], [1, 0, 3], [4, 1, 0], [0, 5, 1]], np.int32)
    coact, load = O.coact_stats(ids, 6)
    assert coact[0, 1] == coact[1, 0] == load[0] == load[1] == 4
    assert coact[0, 1] / np.sqrt(load[0] * load[1]) == 1.0
    assert coact[2, 3] == 0


def test_stats_rejects_bad_ids():
    with pytest.raises(O.OracleError):
        O.coact_stats(np.array([[0, 0]], np.int32), 4)
    with pytest.raises(O.OracleError):
        O.coact_stats(np.array([[0, 4]], np.int32), 4)
    with pytest.raises(O.OracleError):
        O.coact_stats(np.array([[-1, 2]], np.int32), 4)


def test_stats_empty():
    coact, load = O.coact_stats(np.zeros((0, 3), np.int32), 5)
    assert coact.sum() == 0 and load.sum() == 0


# ---------------------------------------------------------------- permutation -------------
def _slots(name, T):
    w = W.make_config(name, T=T)
    r = O.assign(w.N, w.Q, w.S, w.E, w.slot_expert, w.primary_slot, w.topk_ids, w.src_rank, w.seed)
    return w, r


@pytest.mark.parametrize("name,T", [("1", 4096), ("2", 3001), ("3", 2500), ("5", 1500)])
def test_permute_is_the_stable_sort_by_destination(name, T):
    w, r = _slots(name, T)
    x = w.hidden_rows(0, T)[:, :64].copy()
    p = O.permute(r["assigned_slot"], w.D, x)
    flat = r["assigned_slot"].ravel()
    order = np.argsort(flat, kind="stable")                  # library routine
    assert (p["pair_of_row"] == order).all()
    assert (p["row_of_pair"][order] == np.arange(w.P)).all()
    assert (p["dest_counts"] == np.bincount(flat, minlength=w.D)).all()
    assert (p["dest_counts"] == r["slot_load"]).all()        # w_er of Section 3.1
    assert p["dest_offsets"][0] == 0 and p["dest_offsets"][-1] == w.P
    assert (np.diff(p["dest_offsets"].astype(np.int64)) == p["dest_counts"]).all()
    assert (p["send"] == x[order // w.K]).all()
    # rows of one destination hold ascending pair ids (stability)
    for d in range(w.D):
        seg = p["pair_of_row"][p["dest_offsets"][d]:p["dest_offsets"][d + 1]]
        assert (np.diff(seg) > 0).all()
        assert (flat[seg] == d).all()


def test_permute_empty_destinations_and_tiny():
    slots = np.array([[3, 1], [3, 0], [1, 3]], np.int32)       # D = 6, slots 2,4,5 unused
    p = O.permute(slots, 6)
    assert p["dest_counts"].tolist() == [1, 2, 0, 3, 0, 0]
    assert p["dest_offsets"].tolist() == [0, 1, 3, 3, 6, 6, 6]
    assert p["row_of_pair"].tolist() == [3, 1, 4, 0, 2, 5]
    assert p["pair_of_row"].tolist() == [3, 1, 4, 0, 2, 5]
    p0 = O.permute(np.zeros((0, 2), np.int32), 4)
    assert p0["dest_offsets"].tolist() == [0, 0, 0, 0, 0]


def test_permute_rejects_out_of_range_slot():
    with pytest.raises(O.OracleError):
        O.permute(np.array([[0, 4]], np.int32), 4)
    with pytest.raises(O.OracleError):
        O.permute(np.array([[0, -1]], np.int32), 4)


# ---------------------------------------------------------------- combine -----------------
def _setup_combine(name="3", T=300, H=96):
    w, r = _slots(name, T)
    x = w.hidden_rows(0, T)[:, :H].copy()
    p = O.permute(r["assigned_slot"], w.D, x)
    return w, p, x


def test_combine_identity_experts_recover_the_token():
    """Identity experts and gate weights summing to 1: y = x up to fp32 rounding of the sum."""
    w, p, x = _setup_combine()
    y = O.combine(p["send"], p["row_of_pair"], w.gate_w)
    xf = W.f32_from_bf16_bits(x)
    assert np.abs(y - xf).max() <= 4e-6 * max(1.0, np.abs(xf).max())


def test_combine_k1_unit_weight_is_exact_copy():
    w = W.make_custom(257, 8, 1, 40, 2, 2, 3, seed=4)
    r = O.assign(w.N, w.Q, w.S, w.E, w.slot_expert, None, w.topk_ids, w.src_rank, 3)
    x = w.hidden_rows()
    p = O.permute(r["assigned_slot"], w.D, x)
    y = O.combine(p["send"], p["row_of_pair"], np.ones((w.T, 1), np.float32))
    assert (y == W.f32_from_bf16_bits(x)).all()


def test_combine_one_hot_weights_select_one_row():
    w, p, _ = _setup_combine()
    out = w.expert_out_rows()[:, :96].copy()
    g = np.zeros((w.T, w.K), np.float32)
    pick = np.arange(w.T) % w.K
    g[np.arange(w.T), pick] = 1.0
    y = O.combine(out, p["row_of_pair"], g)
    rows = p["row_of_pair"].reshape(w.T, w.K)[np.arange(w.T), pick]
    assert (y == W.f32_from_bf16_bits(out[rows])).all()


def test_combine_matches_float64_sum_within_rounding():
    """Against the real-number definition computed in float64 (independent of summation order)."""
    w, p, _ = _setup_combine(T=400, H=128)
    out = w.expert_out_rows()[:, :128].copy()
    y = O.combine(out, p["row_of_pair"], w.gate_w)
    rows = p["row_of_pair"].reshape(w.T, w.K)
    vals = W.f32_from_bf16_bits(out).astype(np.float64)[rows]          # [T,K,H]
    g = w.gate_w.astype(np.float64)[:, :, None]
    exact = (g * vals).sum(axis=1)
    bound = (w.K + 1) * 2.0 ** -24 * (np.abs(g * vals)).sum(axis=1) + 1e-30
    assert (np.abs(y - exact) <= bound).all()


def test_combine_is_linear_in_the_weights():
    w, p, _ = _setup_combine(T=200, H=64)
    out = w.expert_out_rows()[:, :64].copy()
    g2 = (w.gate_w * np.float32(2.0)).astype(np.float32)       # scaling by 2 is exact in fp32
    y1 = O.combine(out, p["row_of_pair"], w.gate_w)
    y2 = O.combine(out, p["row_of_pair"], g2)
    assert (y2 == 2.0 * y1).all()


def test_combine_token_subset():
    w, p, _ = _setup_combine(T=200, H=64)
    out = w.expert_out_rows()[:, :64].copy()
    y = O.combine(out, p["row_of_pair"], w.gate_w)
    tok = [199, 0, 17, 17, 42]
    ys = O.combine(out, p["row_of_pair"], w.gate_w, tokens=tok)
    assert (ys == y[tok]).all()
