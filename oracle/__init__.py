"""CPU oracle for the Cobalt token-routing path: numpy-facing wrappers over cobalt_oracle.c.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package may import this module; it exists
so that tests, the smoke check and the bench's CPU-baseline leg can compare the CUDA path
with a plain statement of the paper's definitions.  The arithmetic lives in cobalt_oracle.c
(each function cites the passage it follows); this file only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
from typing import Optional, Sequence

import numpy as np

from . import build as _build
from .bruteforce import min_remote_nodes_bruteforce  # noqa: F401
from .dedup import dedup_index, dedup_rows, forward_rows  # noqa: F401
from .epilogue import ema_update, ochiai, rebalance_intra_node  # noqa: F401

_lib = C.CDLL(_build.build())

_i32p = np.ctypeslib.ndpointer(np.int32, flags="C_CONTIGUOUS")
_u32p = np.ctypeslib.ndpointer(np.uint32, flags="C_CONTIGUOUS")
_u16p = np.ctypeslib.ndpointer(np.uint16, flags="C_CONTIGUOUS")
_u8p = np.ctypeslib.ndpointer(np.uint8, flags="C_CONTIGUOUS")
_u64p = np.ctypeslib.ndpointer(np.uint64, flags="C_CONTIGUOUS")
_f32p = np.ctypeslib.ndpointer(np.float32, flags="C_CONTIGUOUS")

_lib.oracle_hash.restype = C.c_uint32
_lib.oracle_hash.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32]
_lib.oracle_hash_index.restype = C.c_uint32
_lib.oracle_hash_index.argtypes = [C.c_uint32, C.c_uint32]
_lib.oracle_layout_tables.restype = C.c_int
_lib.oracle_layout_tables.argtypes = [C.c_int32] * 4 + [_i32p, C.c_void_p, _u32p, _i32p, _i32p, _i32p]
_lib.oracle_coact_stats.restype = C.c_int
_lib.oracle_coact_stats.argtypes = [_i32p, C.c_int64, C.c_int32, C.c_int32, _u32p, _u32p]
_lib.oracle_assign.restype = C.c_int
_lib.oracle_assign.argtypes = [C.c_int32] * 4 + [_i32p, C.c_void_p, _i32p, _i32p, C.c_int64, C.c_int32,
                                                 C.c_uint64, C.c_uint32, _i32p, _u32p, _u8p, _u64p]
_lib.oracle_traffic.restype = C.c_int
_lib.oracle_traffic.argtypes = [C.c_int32] * 4 + [_i32p, _i32p, _i32p, _i32p, C.c_int64, C.c_int32,
                                                  _u8p, _u64p]
_lib.oracle_permute.restype = C.c_int
_lib.oracle_permute.argtypes = [_i32p, C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_int32,
                                C.c_void_p, _u32p, _u32p, _i32p, _i32p]
_lib.oracle_combine.restype = C.c_int
_lib.oracle_combine.argtypes = [_u16p, _i32p, _f32p, C.c_int64, C.c_int32, C.c_int32, C.c_void_p,
                                C.c_int64, _f32p]


_f64p = np.ctypeslib.ndpointer(np.float64, flags="C_CONTIGUOUS")
_lib.oracle_permute_backward.restype = C.c_int
_lib.oracle_permute_backward.argtypes = [_u16p, _i32p, C.c_int64, C.c_int32, C.c_int32, _f64p]
_lib.oracle_combine_backward.restype = C.c_int
_lib.oracle_combine_backward.argtypes = [_u16p, _u16p, _i32p, _f32p, C.c_int64, C.c_int32, C.c_int32, _f64p, _f64p]


class OracleError(ValueError):
    pass


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise OracleError(f"{what}: oracle status {rc}")


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _opt_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def hash32(seed: int, t: int, e: int, stream: int) -> int:
    return int(_lib.oracle_hash(seed & (2**64 - 1), t, e, stream))


def hash_index(x: int, n: int) -> int:
    return int(_lib.oracle_hash_index(x, n))


def layout_tables(N: int, Q: int, S: int, E: int, slot_expert, primary_slot=None):
    """-> dict(nodes_mask [E], r_count [E,N], r_list [E,N,Q], primary [E]); raises on a bad layout."""
    slot_expert = _i32(slot_expert)
    if slot_expert.size != N * Q * S:
        raise OracleError("slot_expert must have N*Q*S entries")
    prim_in = None if primary_slot is None else _i32(primary_slot)
    nodes = np.zeros(E, np.uint32)
    r_count = np.zeros((E, N), np.int32)
    r_list = np.zeros((E, N, Q), np.int32)
    primary = np.zeros(E, np.int32)
    _check(_lib.oracle_layout_tables(N, Q, S, E, slot_expert, _opt_ptr(prim_in), nodes, r_count,
                                     r_list, primary), "layout_tables")
    return dict(nodes_mask=nodes, r_count=r_count, r_list=r_list, primary=primary)


def coact_stats(topk_ids, E: int):
    """-> (coact uint32 [E,E], load uint32 [E])."""
    ids = _i32(topk_ids)
    T, K = ids.shape
    coact = np.zeros((E, E), np.uint32)
    load = np.zeros(E, np.uint32)
    _check(_lib.oracle_coact_stats(ids, T, K, E, coact, load), "coact_stats")
    return coact, load


def assign(N: int, Q: int, S: int, E: int, slot_expert, primary_slot, topk_ids, src_rank, seed: int,
           *, naive: bool = False, round_robin: bool = False):
    """Algorithm 1 (or the naive primary-replica rule; or Algorithm 1 with the round-robin replica pick).

    -> dict(assigned_slot int32 [T,K], slot_load uint32 [D], remote_nodes uint8 [T],
            V int, V_naive int)
    """
    ids = _i32(topk_ids)
    T, K = ids.shape
    slot_expert = _i32(slot_expert)
    src = _i32(src_rank)
    prim_in = None if primary_slot is None else _i32(primary_slot)
    D = N * Q * S
    out = np.zeros((T, K), np.int32)
    slot_load = np.zeros(D, np.uint32)
    remote = np.zeros(T, np.uint8)
    totals = np.zeros(2, np.uint64)
    _check(_lib.oracle_assign(N, Q, S, E, slot_expert, _opt_ptr(prim_in), ids, src, T, K,
                              seed & (2**64 - 1), (1 if naive else 0) | (2 if round_robin else 0), out, slot_load,
                              remote, totals),
           "assign")
    return dict(assigned_slot=out, slot_load=slot_load, remote_nodes=remote,
                V=int(totals[0]), V_naive=int(totals[1]))


def traffic(N: int, Q: int, S: int, E: int, slot_expert, topk_ids, src_rank, assigned_slot):
    """Eq. 1 evaluated from an assignment -> (V, per-token terms uint8 [T])."""
    ids = _i32(topk_ids)
    T, K = ids.shape
    per = np.zeros(T, np.uint8)
    V = np.zeros(1, np.uint64)
    _check(_lib.oracle_traffic(N, Q, S, E, _i32(slot_expert), ids, _i32(src_rank),
                               _i32(assigned_slot).reshape(T, K), T, K, per, V), "traffic")
    return int(V[0]), per


def permute(assigned_slot, D: int, x_bits: Optional[np.ndarray] = None):
    """-> dict(dest_counts [D], dest_offsets [D+1], row_of_pair [P], pair_of_row [P], send [P,H] or None)."""
    slots = _i32(assigned_slot)
    T, K = slots.shape
    P = T * K
    counts = np.zeros(D, np.uint32)
    offsets = np.zeros(D + 1, np.uint32)
    row_of_pair = np.zeros(P, np.int32)
    pair_of_row = np.zeros(P, np.int32)
    send = None
    H = 0
    if x_bits is not None:
        x_bits = np.ascontiguousarray(x_bits, dtype=np.uint16)
        assert x_bits.shape[0] == T
        H = x_bits.shape[1]
        send = np.zeros((P, H), np.uint16)
    _check(_lib.oracle_permute(slots, T, K, D, _opt_ptr(x_bits), H, _opt_ptr(send), counts, offsets,
                               row_of_pair, pair_of_row), "permute")
    return dict(dest_counts=counts, dest_offsets=offsets, row_of_pair=row_of_pair,
                pair_of_row=pair_of_row, send=send)


def combine(expert_out_bits, row_of_pair, gate_w, tokens: Optional[Sequence[int]] = None) -> np.ndarray:
    """fp32 y [T,H] (or [len(tokens),H]) = gate-weighted sum of the K expert rows of each token."""
    out = np.ascontiguousarray(expert_out_bits, dtype=np.uint16)
    w = np.ascontiguousarray(gate_w, dtype=np.float32)
    T, K = w.shape
    H = out.shape[1]
    rop = _i32(row_of_pair).reshape(-1)
    tok = None if tokens is None else np.ascontiguousarray(tokens, dtype=np.int64)
    n = T if tok is None else tok.size
    y = np.zeros((n, H), np.float32)
    _check(_lib.oracle_combine(out, rop, w, T, K, H, _opt_ptr(tok), n, y), "combine")
    return y


def permute_backward(grad_send_bits, row_of_pair, T: int, K: int) -> np.ndarray:
    """float64 grad_x [T,H] = sum over a token's K send rows of grad_send."""
    g = np.ascontiguousarray(grad_send_bits, dtype=np.uint16)
    H = g.shape[1]
    out = np.zeros((T, H), np.float64)
    _check(_lib.oracle_permute_backward(g, _i32(row_of_pair).reshape(-1), T, K, H, out), "permute_backward")
    return out


def combine_backward(grad_y_bits, expert_out_bits, row_of_pair, gate_w):
    """-> (float64 grad_expert_out [P,H], float64 grad_gate_w [T,K])."""
    gy = np.ascontiguousarray(grad_y_bits, dtype=np.uint16)
    out = np.ascontiguousarray(expert_out_bits, dtype=np.uint16)
    w = np.ascontiguousarray(gate_w, dtype=np.float32)
    T, K = w.shape
    H = gy.shape[1]
    grad_out = np.zeros((T * K, H), np.float64)
    grad_w = np.zeros((T, K), np.float64)
    _check(_lib.oracle_combine_backward(gy, out, _i32(row_of_pair).reshape(-1), w, T, K, H, grad_out, grad_w),
           "combine_backward")
    return grad_out, grad_w
