"""The library's Stage-2 rebalancer is host code: compared with the oracle here, without a GPU."""
import numpy as np
import pytest

import oracle as O
import workloads as W


@pytest.fixture(scope="module")
def cb():
    from paper_2609_36959_b200 import build
    build.build()
    import paper_2609_36959_b200.binding as binding
    return binding


@pytest.mark.parametrize("name", ["1", "1a", "2", "3", "4", "5"])
def test_rebalancer_matches_the_oracle_on_configs(cb, name):
    w = W.make_config(name, T=3000)
    r = O.assign(w.N, w.Q, w.S, w.E, w.slot_expert, w.primary_slot, w.topk_ids, w.src_rank, w.seed)
    ema = (0.7 * r["slot_load"] + 0.3 * np.roll(r["slot_load"], 1) * (w.slot_expert >= 0)).astype(np.float32)
    new, moved, kept = cb.rebalance_intra_node(w.N, w.Q, w.S, w.E, w.slot_expert.tolist(), ema.tolist())
    ref_new, ref_moved, ref_kept = O.rebalance_intra_node(w.N, w.Q, w.S, w.slot_expert, ema)
    assert new == ref_new.tolist() and moved == ref_moved.tolist() and kept == len(ref_kept)
    assert cb.layout_check(w.N, w.Q, w.S, w.E, new) == cb.OK          # the result is a valid layout


def test_rebalancer_hand_examples_and_dead_end(cb):
    assert cb.rebalance_intra_node(1, 2, 2, 4, [0, 1, 2, 3], [10, 7, 5, 3]) == ([0, 3, 1, 2], [0, 3, 1, 2], 0)
    assert cb.rebalance_intra_node(1, 2, 3, 2, [1, 0, -1, 0, -1, -1], [10, 5, 0, 4, 0, 0]) == (
        [1, 0, -1, 0, -1, -1], [0, 3, -1, 1, -1, -1], 0)
    assert cb.rebalance_intra_node(1, 2, 2, 3, [0, 1, 2, 0], [10, 9, 8, 1]) == ([0, 1, 2, 0], [0, 1, 2, 3], 1)
    with pytest.raises(cb.CobaltError):
        cb.rebalance_intra_node(1, 2, 2, 3, [0, 0, 2, 1], [1, 1, 1, 1])      # expert twice on a rank


def test_rebalancer_with_ties_and_empty_slots(cb):
    rng = np.random.default_rng(2)
    for trial in range(50):
        N, Q, S, E = 2, 3, 3, 7
        w = W.make_custom(50, E, 2, 8, N, Q, S, seed=trial, n_empty=int(rng.integers(0, 4)))
        load = rng.integers(0, 4, N * Q * S).astype(np.float32) * (w.slot_expert >= 0)   # many ties
        new, moved, kept = cb.rebalance_intra_node(N, Q, S, E, w.slot_expert.tolist(), load.tolist())
        ref_new, ref_moved, ref_kept = O.rebalance_intra_node(N, Q, S, w.slot_expert, load)
        assert new == ref_new.tolist() and moved == ref_moved.tolist() and kept == len(ref_kept)


@pytest.mark.parametrize("bad", [float("nan"), float("inf"), -1.0])
def test_rebalancer_refuses_loads_that_cannot_be_ordered(cb, bad):
    """A NaN load would leave the longest-first sort without a strict weak order: such inputs are
    refused as invalid arguments instead (empty slots may hold anything)."""
    with pytest.raises(cb.CobaltError) as err:
        cb.rebalance_intra_node(1, 2, 2, 4, [0, 1, 2, 3], [10, bad, 5, 3])
    assert err.value.status == cb.ERR_INVALID_ARG
    assert cb.rebalance_intra_node(1, 2, 2, 3, [0, 1, 2, -1], [3, 2, 1, bad])[2] == 0
