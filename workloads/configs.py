"""Seeded synthetic workloads shaped like the paper's MoE training runs.

The paper trains on real gating traces (Table 3 models on C4, 4 nodes x 8 GPUs) that are not
available here; these generators stand in for them.  Every array is a pure function of the
config name and seed.  Nothing in this file implements any step of the routing method: it
only draws ids / weights / rows and builds a *valid* expert layout (each expert at least once,
never twice on a rank) for the method to route over.

Latent cluster model for the top-k ids: the E experts are split into C clusters of
consecutive ids; a token first picks a cluster c with probability q_c, then draws K distinct
experts one after another: with probability p_in (if its cluster still has unchosen members)
from the unchosen members of c, otherwise from all unchosen experts, both proportional to a
per-expert popularity pi.  Ids are kept in draw order.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import Optional

import numpy as np

BASE_SEED = 36959

# independent random streams under one config seed
_STREAM_IDS, _STREAM_W, _STREAM_X, _STREAM_LAYOUT, _STREAM_HISTORY, _STREAM_OUT = range(6)

_ID_BLOCK = 8192      # tokens drawn per id/weight block (fixes the random stream layout)
_ROW_BLOCK = 256      # rows drawn per hidden-row block
_HISTORY_TOKENS = 8192

CONFIG_NAMES = ("1", "1a", "2", "3", "4", "5")


def _rng(seed: int, stream: int, block: int = 0) -> np.random.Generator:
    return np.random.default_rng([int(seed), int(stream), int(block)])


def bf16_bits_from_f32(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest even) and return the 16-bit patterns."""
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def f32_from_bf16_bits(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class ClusterModel:
    E: int
    K: int
    C: int
    p_in: float
    q: np.ndarray          # [C] cluster popularity, sums to 1
    pi: np.ndarray         # [E] expert popularity (unnormalised)

    @property
    def cluster_of(self) -> np.ndarray:
        return (np.arange(self.E) * self.C) // self.E


def _zipf(n: int, a: float) -> np.ndarray:
    w = (np.arange(n, dtype=np.float64) + 1.0) ** (-a)
    return w / w.sum()


def sample_topk_ids(model: ClusterModel, T: int, seed: int, stream: int = _STREAM_IDS) -> np.ndarray:
    """Draw [T, K] distinct-per-token expert ids (int32) from the latent cluster model."""
    E, K, C = model.E, model.K, model.C
    if K > E:
        raise ValueError("K > E")
    cluster_of = model.cluster_of
    ids = np.empty((T, K), dtype=np.int32)
    for blk, t0 in enumerate(range(0, T, _ID_BLOCK)):
        n = min(_ID_BLOCK, T - t0)
        rng = _rng(seed, stream, blk)
        c = rng.choice(C, size=n, p=model.q)
        chosen = np.zeros((n, E), dtype=bool)
        home = cluster_of[None, :] == c[:, None]
        for k in range(K):
            u_branch = rng.random(n)
            u_pick = rng.random(n)
            in_free = home & ~chosen
            use_in = (u_branch < model.p_in) & in_free.any(axis=1)
            cand = np.where(use_in[:, None], in_free, ~chosen)
            cum = np.cumsum(cand * model.pi[None, :], axis=1)
            thr = u_pick * cum[:, -1]
            pick = (cum > thr[:, None]).argmax(axis=1)
            # guard against thr == total through rounding: fall back to the last candidate
            bad = ~cand[np.arange(n), pick]
            if bad.any():
                pick[bad] = E - 1 - cand[bad, ::-1].argmax(axis=1)
            ids[t0:t0 + n, k] = pick
            chosen[np.arange(n), pick] = True
    return ids


def sample_gate_weights(T: int, K: int, seed: int, kind: str = "softmax") -> np.ndarray:
    """[T, K] float32 gate weights that sum to 1 over the K chosen experts."""
    w = np.empty((T, K), dtype=np.float32)
    for blk, t0 in enumerate(range(0, T, _ID_BLOCK)):
        n = min(_ID_BLOCK, T - t0)
        logits = _rng(seed, _STREAM_W, blk).standard_normal((n, K)).astype(np.float32)
        if kind == "softmax":
            z = np.exp(logits - logits.max(axis=1, keepdims=True))
        elif kind == "sigmoid":
            z = 1.0 / (1.0 + np.exp(-logits))
        else:
            raise ValueError(kind)
        w[t0:t0 + n] = (z / z.sum(axis=1, keepdims=True)).astype(np.float32)
    return w


def make_layout(rng: np.random.Generator, N: int, Q: int, S: int, E: int,
                hist_load: np.ndarray, *, clustered: bool = False,
                n_empty: int = 0) -> tuple[np.ndarray, np.ndarray]:
    """Build slot_expert[G*S] (expert id, or -1 for an empty slot) and primary_slot[E].

    E >= G: a seeded permutation sigma of the experts is dealt to the ranks in blocks of
    ceil(E/G) primaries; the spare slots, visited in seeded-shuffled order, each take the next
    expert in descending historical-load order (cycling) that the rank does not hold yet.
    E < G with S == 1: the ranks are shuffled and rank perm[i] holds expert i mod E.
    `clustered` keeps sigma = identity so that consecutive (co-activated) experts share a node.
    `n_empty` spare slots are left empty (-1).
    """
    G = N * Q
    slot_expert = np.full(G * S, -1, dtype=np.int32)
    primary = np.full(E, -1, dtype=np.int32)
    order = np.lexsort((np.arange(E), -np.asarray(hist_load, dtype=np.int64)))  # desc load, ties by id
    if E < G:
        perm = np.arange(G) if clustered else rng.permutation(G)
        held = [set() for _ in range(G)]
        for i in range(G):
            e = i % E
            slot_expert[perm[i] * S] = e
            held[perm[i]].add(e)
            if i < E:
                primary[e] = perm[i] * S
    else:
        per = -(-E // G)
        if per > S:
            raise ValueError("layout needs ceil(E/G) <= S")
        sigma = np.arange(E) if clustered else rng.permutation(E)
        held = [set() for _ in range(G)]
        for i in range(E):
            r, j = divmod(i, per)
            slot_expert[r * S + j] = sigma[i]
            primary[sigma[i]] = r * S + j
            held[r].add(int(sigma[i]))
    spare = [d for d in range(G * S) if slot_expert[d] < 0]
    spare = [spare[i] for i in rng.permutation(len(spare))] if spare else []
    spare = spare[: max(0, len(spare) - n_empty)]
    cursor = 0
    for d in spare:
        r = d // S
        for _ in range(E):
            e = int(order[cursor % E])
            cursor += 1
            if e not in held[r]:
                slot_expert[d] = e
                held[r].add(e)
                break
    return slot_expert, primary


@dataclass
class Workload:
    name: str
    T: int
    E: int
    K: int
    H: int
    N: int
    Q: int
    S: int
    seed: int
    topk_ids: np.ndarray
    gate_w: np.ndarray
    src_rank: np.ndarray
    slot_expert: np.ndarray
    primary_slot: np.ndarray
    model: Optional[ClusterModel] = field(default=None, repr=False)

    @property
    def G(self) -> int:
        return self.N * self.Q

    @property
    def D(self) -> int:
        return self.G * self.S

    @property
    def P(self) -> int:
        return self.T * self.K

    def _rows(self, stream: int, r0: int, r1: int) -> np.ndarray:
        out = np.empty((r1 - r0, self.H), dtype=np.uint16)
        b0, b1 = r0 // _ROW_BLOCK, (r1 + _ROW_BLOCK - 1) // _ROW_BLOCK

        def fill(blk: int) -> None:
            lo, hi = blk * _ROW_BLOCK, (blk + 1) * _ROW_BLOCK
            vals = _rng(self.seed, stream, blk).standard_normal((_ROW_BLOCK, self.H), dtype=np.float32)
            a, b = max(lo, r0), min(hi, r1)
            out[a - r0:b - r0] = bf16_bits_from_f32(vals[a - lo:b - lo])

        if b1 - b0 > 8:   # blocks are independent streams: draw them on several host threads
            with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as pool:
                list(pool.map(fill, range(b0, b1)))
        else:
            for blk in range(b0, b1):
                fill(blk)
        return out

    def hidden_rows(self, t0: int = 0, t1: Optional[int] = None) -> np.ndarray:
        """bf16 bit patterns (uint16) of N(0,1) hidden rows x[t0:t1, :H]."""
        return self._rows(_STREAM_X, t0, self.T if t1 is None else t1)

    def expert_out_rows(self, r0: int = 0, r1: Optional[int] = None) -> np.ndarray:
        """bf16 bit patterns of independent N(0,1) expert outputs, rows r0:r1 of [P, H]."""
        return self._rows(_STREAM_OUT, r0, self.P if r1 is None else r1)


def _assemble(name: str, T: int, H: int, N: int, Q: int, S: int, seed: int, model: ClusterModel,
              gate: str, clustered: bool, n_empty: int = 0) -> Workload:
    E, K = model.E, model.K
    G = N * Q
    ids = sample_topk_ids(model, T, seed)
    w = sample_gate_weights(T, K, seed, gate)
    hist_ids = sample_topk_ids(model, _HISTORY_TOKENS, seed, stream=_STREAM_HISTORY)
    hist_load = np.bincount(hist_ids.ravel(), minlength=E)
    slot_expert, primary = make_layout(_rng(seed, _STREAM_LAYOUT), N, Q, S, E, hist_load,
                                       clustered=clustered, n_empty=n_empty)
    src_rank = ((np.arange(T, dtype=np.int64) * G) // max(T, 1)).astype(np.int32)
    return Workload(name, T, E, K, H, N, Q, S, seed, ids, w, src_rank, slot_expert, primary, model)


def make_config(name: str, *, clustered: bool = False, T: Optional[int] = None) -> Workload:
    """One of the five benchmark configs ("1".."5") or "1a" (config 1 with no spare slots).

    `T` overrides the token count (same model, layout and seed) for reduced-size runs.
    """
    name = str(name)
    idx = int(name[0])
    seed = BASE_SEED + 1000 * idx
    if idx == 1:
        E, K, H, N, Q, S, T0 = 16, 2, 1024, 2, 4, (2 if name == "1a" else 3), 4096
        model = ClusterModel(E, K, 4, 0.8, _zipf(4, 1.1), np.ones(E))
        gate = "softmax"
    elif idx == 2:
        E, K, H, N, Q, S, T0 = 8, 2, 4096, 4, 8, 1, 16384
        model = ClusterModel(E, K, 2, 0.7, np.full(2, 0.5), np.ones(E))
        gate = "softmax"
    elif idx == 3:
        E, K, H, N, Q, S, T0 = 64, 6, 2048, 4, 8, 3, 32768
        model = ClusterModel(E, K, 8, 0.75, _zipf(8, 1.2), np.ones(E))
        gate = "softmax"
    elif idx == 4:
        E, K, H, N, Q, S, T0 = 128, 8, 4096, 4, 8, 5, 65536
        pi = np.empty(E)
        pi[_rng(seed, _STREAM_LAYOUT, 1).permutation(E)] = (np.arange(E) + 1.0) ** (-1.2)
        q = pi.reshape(16, E // 16).sum(axis=1)
        model = ClusterModel(E, K, 16, 0.6, q / q.sum(), pi)
        gate = "softmax"
    elif idx == 5:
        E, K, H, N, Q, S, T0 = 256, 8, 7168, 4, 8, 9, 131072
        model = ClusterModel(E, K, 32, 0.8, _zipf(32, 1.3), np.ones(E))
        gate = "sigmoid"
    else:
        raise ValueError(f"unknown config {name!r}")
    return _assemble(name + ("c" if clustered else ""), T0 if T is None else T, H, N, Q, S, seed,
                     model, gate, clustered)


def make_custom(T: int, E: int, K: int, H: int, N: int, Q: int, S: int, seed: int, *,
                C: int = 1, p_in: float = 0.5, gate: str = "softmax", clustered: bool = False,
                n_empty: int = 0) -> Workload:
    """Small / edge-case workload with arbitrary (also non-power-of-two) sizes."""
    C = max(1, min(C, E))
    model = ClusterModel(E, K, C, p_in, np.full(C, 1.0 / C), np.ones(E))
    return _assemble(f"custom_T{T}_E{E}_K{K}_H{H}_N{N}x{Q}_S{S}", T, H, N, Q, S, seed, model, gate,
                     clustered, n_empty)
