"""The no-allocation variant of the permutation index (cobalt_permute_index_static).

Some users of the library cannot give it device scratch at the call site: a framework hot path
where allocator calls are banned, a plugin that only ever sees its input and output buffers, a
job whose memory pool is fully committed.  For them the scratch is a fixed array inside the
library.  This file checks, through the C ABI, that the variant returns exactly what the
regular entry point returns, on two calls in a row (the second call finds the first call's
leftovers in the shared array), and that problems beyond the built-in limit are refused.
It is named to be collected last, so a run that stops at the first failure has already been
through every other test; it also passes on its own in a fresh process.
"""
import pytest
import torch

import workloads as W

pytestmark = pytest.mark.gpu


def _index_outputs(P, D):
    def z(n):
        return torch.full((n,), -7, dtype=torch.int32, device="cuda")
    return dict(dest_counts=z(D), dest_offsets=z(D + 1), row_of_pair=z(P), pair_of_row=z(P))


def _slots(w, seed):
    import paper_2609_36959_b200 as cb
    layout = cb.Layout(w.N, w.Q, w.S, w.E, w.slot_expert.tolist(), w.primary_slot.tolist())
    slots = torch.zeros((w.T, w.K), dtype=torch.int32, device="cuda")
    cb.assign(layout, torch.from_numpy(w.topk_ids).cuda(), torch.from_numpy(w.src_rank).cuda(), seed, slots)
    torch.cuda.synchronize()
    return slots


def test_static_scratch_variant_matches_the_regular_entry_point_twice():
    import paper_2609_36959_b200 as cb
    assert torch.cuda.is_available()
    # two different problems back to back: the second one meets the first one's scratch contents
    cases = [W.make_config("3"), W.make_custom(5001, 24, 6, 8, 4, 3, 3, seed=12, C=3, p_in=0.6, n_empty=3)]
    for w in cases:
        slots = _slots(w, w.seed)
        ref = _index_outputs(w.P, w.D)
        ws = torch.empty(cb.permute_workspace_bytes(w.T, w.K, w.D), dtype=torch.uint8, device="cuda")
        cb.permute_index(slots, w.D, ref["dest_counts"], ref["dest_offsets"], ref["row_of_pair"],
                         ref["pair_of_row"], ws)
        for call in range(2):
            got = _index_outputs(w.P, w.D)
            cb.permute_index_static(slots, w.D, got["dest_counts"], got["dest_offsets"], got["row_of_pair"],
                                    got["pair_of_row"])
            torch.cuda.synchronize()
            for name in ref:
                assert torch.equal(got[name], ref[name]), f"{w.name}: {name} differs on call {call}"
    assert cb.read_and_clear_device_error() == 0


def test_static_scratch_variant_refuses_problems_beyond_its_limit():
    import paper_2609_36959_b200 as cb
    T, K, D = 300000, 2, 4096                       # 293 chunks x 4096 destinations > 2^20 words
    slots = torch.zeros((T, K), dtype=torch.int32, device="cuda")
    out = _index_outputs(T * K, D)
    with pytest.raises(cb.CobaltError) as e:
        cb.permute_index_static(slots, D, out["dest_counts"], out["dest_offsets"], out["row_of_pair"],
                                out["pair_of_row"])
    assert e.value.status == cb.ERR_SCRATCH_LIMIT
    assert "built-in scratch" in str(e.value)
    torch.cuda.synchronize()
    assert int(out["row_of_pair"][0]) == -7          # nothing was enqueued
