"""Exhaustive per-token minimum of Eq. 1 (tiny inputs only).  TEST INFRASTRUCTURE ONLY.

For one token, every way of choosing a replica slot for each selected expert is enumerated
(the product over e in D_t of all slots holding e) and the smallest number of distinct remote
nodes reached is returned.  Nothing here knows about bitmasks, set covers or Algorithm 1:
it is the definition of "fewest remote nodes" written out, used to pin Algorithm 1's result.
"""
from __future__ import annotations

import itertools
from typing import Sequence


def min_remote_nodes_bruteforce(slot_expert: Sequence[int], S: int, Q: int, experts: Sequence[int],
                                src_rank: int) -> int:
    src_node = src_rank // Q
    choices = []
    for e in experts:
        slots = [d for d, held in enumerate(slot_expert) if held == e]
        if not slots:
            raise ValueError(f"expert {e} has no replica")
        choices.append(slots)
    best = None
    for combo in itertools.product(*choices):
        nodes = {d // (S * Q) for d in combo}
        nodes.discard(src_node)
        if best is None or len(nodes) < best:
            best = len(nodes)
    return 0 if best is None else best
