"""Pins for the oracle's statistics epilogue and Stage-2 rebalancer (CPU only)."""
import itertools

import numpy as np
import pytest

import oracle as O
import workloads as W


# ---------------------------------------------------------------- Ochiai ------------------
def test_ochiai_matches_the_set_definition():
    """|A n B| / sqrt(|A||B|) computed from the token sets themselves (footnote of Section 1)."""
    w = W.make_config("3", T=3000)
    coact, load = O.coact_stats(w.topk_ids, w.E)
    och = O.ochiai(coact)
    sets = [set(np.nonzero((w.topk_ids == e).any(axis=1))[0].tolist()) for e in range(w.E)]
    rng = np.random.default_rng(0)
    for i, j in rng.integers(0, w.E, size=(200, 2)):
        a, b = sets[i], sets[j]
        ref = len(a & b) / np.sqrt(len(a) * len(b)) if a and b else 0.0
        assert och[i, j] == pytest.approx(ref, abs=1e-15)
    assert np.allclose(np.diag(och)[load > 0], 1.0)
    assert och.min() >= 0 and och.max() <= 1 + 1e-12 and np.allclose(och, och.T)


def test_ochiai_fig1_tokens_and_unused_expert(fig1):
    ids = np.array([tk["ids"] for tk in fig1["tokens"]], np.int32)
    coact, _ = O.coact_stats(ids, 5)                    # expert 4 is never selected
    och = O.ochiai(coact)
    assert np.allclose(och[:4, :4][~np.eye(4, dtype=bool)], fig1["ochiai_offdiag"])
    assert (och[4] == 0).all() and (och[:, 4] == 0).all()


# ---------------------------------------------------------------- EMA ---------------------
def test_ema_closed_form_for_a_constant_input():
    x = np.array([4.0, 0.0, 10.0])
    ema = np.array([1.0, 2.0, 3.0])
    beta = 0.9
    cur = ema.copy()
    for n in range(1, 30):
        cur = O.ema_update(cur, x, beta)
        assert np.allclose(cur, x * (1 - beta ** n) + beta ** n * ema, rtol=1e-12)
    assert np.allclose(O.ema_update(ema, x, 0.0), x) and np.allclose(O.ema_update(ema, x, 1.0), ema)


# ---------------------------------------------------------------- rebalancer --------------
def _check_constraints(N, Q, S, old, new, moved):
    old = np.asarray(old)
    for n in range(N):
        lo, hi = n * Q * S, (n + 1) * Q * S
        assert sorted(old[lo:hi][old[lo:hi] >= 0].tolist()) == sorted(new[lo:hi][new[lo:hi] >= 0].tolist())
        for q in range(Q):
            held = new[lo + q * S: lo + (q + 1) * S]
            held = held[held >= 0]
            assert len(set(held.tolist())) == len(held) <= S
    for d, src in enumerate(moved):
        if new[d] >= 0:
            assert lo_node(src, Q, S) == lo_node(d, Q, S) and old[src] == new[d]
        else:
            assert src == -1
    used = moved[moved >= 0]
    assert len(set(used.tolist())) == len(used)          # every old replica lands exactly once


def lo_node(d, Q, S):
    return d // (Q * S)


def test_rebalance_hand_example_longest_first():
    # one node, 2 ranks x 2 slots: a(10) b(7) on rank 0, c(5) d(3) on rank 1
    # greedy: a -> r0 (10); b -> r1 (7); c -> r1 (12); d -> r0 (13): rank loads 13 / 12 instead of 17 / 8
    new, moved, kept = O.rebalance_intra_node(1, 2, 2, [0, 1, 2, 3], [10, 7, 5, 3])
    assert new.tolist() == [0, 3, 1, 2] and moved.tolist() == [0, 3, 1, 2] and kept == []


def test_rebalance_same_expert_never_twice_on_a_rank():
    # b(10) a(5) a'(4): a' would prefer rank 1 (load 5) but it already holds expert a
    slot = [1, 0, -1, 0, -1, -1]                         # 1 node, 2 ranks, S = 3; old: r0 {b, a}, r1 {a'}
    new, moved, kept = O.rebalance_intra_node(1, 2, 3, slot, [10, 5, 0, 4, 0, 0])
    # sorted: b(10) -> r0; a(5, old slot 1) -> r1; a'(4, old slot 3) -> not r1 (holds a) -> r0
    assert new.tolist() == [1, 0, -1, 0, -1, -1]
    assert moved.tolist() == [0, 3, -1, 1, -1, -1]
    assert kept == []


def test_rebalance_dead_end_keeps_the_node():
    # 2 ranks x 2 slots, a(10) b(9) c(8) a'(1): a -> r0, b -> r1, c -> r1 (now full), a' cannot go to r0
    # (holds a) nor to r1 (full): the node keeps its old placement
    slot = [0, 1, 2, 0]                                   # r0 {a, b}, r1 {c, a}
    new, moved, kept = O.rebalance_intra_node(1, 2, 2, slot, [10, 9, 8, 1])
    assert kept == [0] and new.tolist() == slot and moved.tolist() == [0, 1, 2, 3]


@pytest.mark.parametrize("name", ["1", "3", "5"])
def test_rebalance_constraints_and_balance_on_configs(name):
    w = W.make_config(name, T=4000)
    r = O.assign(w.N, w.Q, w.S, w.E, w.slot_expert, w.primary_slot, w.topk_ids, w.src_rank, w.seed)
    load = r["slot_load"].astype(np.float64)
    new, moved, kept = O.rebalance_intra_node(w.N, w.Q, w.S, w.slot_expert, load)
    _check_constraints(w.N, w.Q, w.S, w.slot_expert, new, moved)
    old_rank = load.reshape(w.G, w.S).sum(axis=1).reshape(w.N, w.Q)
    new_load = np.where(moved >= 0, load[np.maximum(moved, 0)], 0.0)
    new_rank = new_load.reshape(w.G, w.S).sum(axis=1).reshape(w.N, w.Q)
    assert np.allclose(old_rank.sum(axis=1), new_rank.sum(axis=1))      # work stays on its node
    for n in range(w.N):
        if n not in kept:
            # longest-first list scheduling: max <= mean + largest item
            assert new_rank[n].max() <= new_rank[n].mean() + load[n * w.Q * w.S:(n + 1) * w.Q * w.S].max() + 1e-9


def test_rebalance_within_four_thirds_of_the_optimum_when_unconstrained():
    """With distinct experts and room to spare the greedy is plain LPT: max <= (4/3 - 1/(3Q)) OPT."""
    rng = np.random.default_rng(4)
    Q = 3
    for trial in range(30):
        n_rep = int(rng.integers(4, 8))
        S = n_rep
        loads = rng.integers(1, 30, n_rep).astype(float)
        slot = np.full(Q * S, -1)
        slot[:n_rep] = np.arange(n_rep)                   # all on rank 0 to start with
        ld = np.zeros(Q * S)
        ld[:n_rep] = loads
        new, moved, kept = O.rebalance_intra_node(1, Q, S, slot, ld)
        assert kept == []
        got = np.where(moved >= 0, ld[np.maximum(moved, 0)], 0.0).reshape(Q, S).sum(axis=1).max()
        best = min(max(sum(loads[i] for i in range(n_rep) if a[i] == q) for q in range(Q))
                   for a in itertools.product(range(Q), repeat=n_rep))
        assert got <= (4.0 / 3.0 - 1.0 / (3 * Q)) * best + 1e-9
