"""ctypes binding of libcobalt.so: same names as the C ABI, argument marshalling only.

Every step of the routing path runs in the library's CUDA kernels.  torch is used for device
memory and streams: tensors are passed as raw device pointers and the current torch stream is
the stream the kernels are enqueued on.  There is no CPU fallback: if the shared library is
missing or a call fails, a CobaltError is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libcobalt.so")

OK = 0
ERR_INVALID_ARG = -1
ERR_WORKSPACE_TOO_SMALL = -2
ERR_UNSUPPORTED = -3
ERR_CUDA = -4
ERR_SCRATCH_LIMIT = -5
ERR_HOST_ALLOC = -6
STATIC_SCRATCH_WORDS = 1 << 20

DEVERR_BAD_EXPERT_ID = 0x1
DEVERR_DUPLICATE_ID = 0x2
DEVERR_BAD_SRC_RANK = 0x4
DEVERR_BAD_SLOT = 0x8
DEVERR_WAIT_TIMEOUT = 0x10

STATS_ACCUMULATE = 0x1
ASSIGN_NAIVE = 0x1
ASSIGN_ROUND_ROBIN = 0x2
SEED_ON_DEVICE = 0x4
STATS_TILE16 = 0x10
STATS_TILE32 = 0x20
ROUTE_SEPARATE_KERNELS = 0x40
EMA_INITIALISE = 0x1
IMPL_VECTOR = 0x100
IMPL_BULK = 0x200

# every symbol include/cobalt.h declares
EXPORTS = (
    "cobalt_status_string", "cobalt_version", "cobalt_last_cuda_error",
    "cobalt_layout_check", "cobalt_layout_create", "cobalt_layout_destroy", "cobalt_layout_num_dests",
    "cobalt_coact_stats_workspace_bytes", "cobalt_coact_stats",
    "cobalt_assign_workspace_bytes", "cobalt_assign",
    "cobalt_permute_workspace_bytes", "cobalt_permute_index", "cobalt_permute_rows", "cobalt_permute",
    "cobalt_permute_index_static", "cobalt_permute_rows_block", "cobalt_combine_block",
    "cobalt_route_index_workspace_bytes", "cobalt_route_index",
    "cobalt_permute_backward", "cobalt_combine_backward",
    "cobalt_ema_update", "cobalt_ochiai", "cobalt_rebalance_intra_node",
    "cobalt_dedup_workspace_bytes", "cobalt_dedup_index", "cobalt_forward_rows",
    "cobalt_combine", "cobalt_read_and_clear_device_error",
)


class CobaltError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} (status {status}, cuda error {last_cuda_error()})")


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2609_36959_b200.build` "
            "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, u32, u64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_uint64, C.c_size_t
    sig = {
        "cobalt_status_string": (C.c_char_p, [C.c_int]),
        "cobalt_version": (C.c_int, []),
        "cobalt_last_cuda_error": (C.c_int, []),
        "cobalt_layout_check": (C.c_int, [i32, i32, i32, i32, vp, vp]),
        "cobalt_layout_create": (C.c_int, [C.POINTER(vp), i32, i32, i32, i32, vp, vp]),
        "cobalt_layout_destroy": (C.c_int, [vp]),
        "cobalt_layout_num_dests": (i32, [vp]),
        "cobalt_coact_stats_workspace_bytes": (sz, [i64, i32, i32]),
        "cobalt_coact_stats": (C.c_int, [vp, i64, i32, i32, vp, vp, u32, vp, sz, vp]),
        "cobalt_assign_workspace_bytes": (sz, [vp, i64, i32]),
        "cobalt_assign": (C.c_int, [vp, vp, vp, i32, i64, i32, u64, vp, vp, vp, vp, u32, vp, sz, vp]),
        "cobalt_permute_workspace_bytes": (sz, [i64, i32, i32]),
        "cobalt_permute_index": (C.c_int, [vp, i64, i32, i32, vp, vp, vp, vp, vp, sz, vp]),
        "cobalt_permute_index_static": (C.c_int, [vp, i64, i32, i32, vp, vp, vp, vp, vp]),
        "cobalt_permute_rows": (C.c_int, [vp, vp, i64, i32, i32, vp, u32, vp]),
        "cobalt_permute": (C.c_int, [vp, i64, i32, i32, vp, i32, vp, vp, vp, vp, vp, u32, vp, sz, vp]),
        "cobalt_combine": (C.c_int, [vp, vp, vp, i64, i32, i32, vp, u32, vp]),
        "cobalt_route_index_workspace_bytes": (sz, [vp, i64, i32]),
        "cobalt_route_index": (C.c_int, [vp, vp, vp, i32, i64, i32, u64, vp, vp, vp, vp, vp, vp, vp, vp, vp, u32, vp,
                                         sz, vp]),
        "cobalt_permute_backward": (C.c_int, [vp, vp, i64, i32, i32, vp, u32, vp]),
        "cobalt_combine_backward": (C.c_int, [vp, vp, vp, vp, i64, i32, i32, vp, vp, u32, vp]),
        "cobalt_ema_update": (C.c_int, [vp, vp, i64, C.c_float, u32, vp]),
        "cobalt_ochiai": (C.c_int, [vp, i32, vp, vp]),
        "cobalt_rebalance_intra_node": (C.c_int, [i32, i32, i32, i32, vp, vp, vp, vp, vp]),
        "cobalt_dedup_workspace_bytes": (sz, [i64, i32, i32]),
        "cobalt_dedup_index": (C.c_int, [vp, vp, i32, i64, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, sz, vp]),
        "cobalt_forward_rows": (C.c_int, [vp, vp, vp, i64, i32, vp, i64, i64, vp]),
        "cobalt_permute_rows_block": (C.c_int, [vp, vp, i64, i32, i32, vp, i64, u32, vp]),
        "cobalt_combine_block": (C.c_int, [vp, vp, vp, i64, i32, i32, vp, i64, u32, vp]),
        "cobalt_read_and_clear_device_error": (C.c_int, [C.POINTER(u32), vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    return lib


_lib = _load()


def status_string(status: int) -> str:
    return _lib.cobalt_status_string(status).decode()


def version() -> int:
    return _lib.cobalt_version()


def last_cuda_error() -> int:
    return _lib.cobalt_last_cuda_error()


def _check(status: int, what: str) -> None:
    if status != OK:
        raise CobaltError(status, what)


def _ptr(t: Optional[torch.Tensor], dtype: Optional[torch.dtype] = None, what: str = "tensor") -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise TypeError(f"{what} must be a CUDA tensor")
    if not t.is_contiguous():
        raise TypeError(f"{what} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{what} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream() -> int:
    """Handle of torch's current stream on the current device (the raw query costs a fraction of a
    microsecond; building a torch.cuda.Stream object for it costs about three)."""
    if _raw_stream is not None:
        return _raw_stream(torch.cuda.current_device())
    return torch.cuda.current_stream().cuda_stream


def _seed_arg(seed, flags: int):
    """A Python int is passed by value; a one-element int64 CUDA tensor is passed by address and read
    by the kernel when it runs (COBALT_SEED_ON_DEVICE), which lets a captured graph be replayed with
    another seed."""
    if isinstance(seed, torch.Tensor):
        if seed.numel() != 1:
            raise TypeError("a seed tensor must have one element")
        return _ptr(seed, torch.int64, "seed"), flags | SEED_ON_DEVICE
    return seed & (2**64 - 1), flags


def _host_i32(a) -> "C.Array":
    vals = [int(v) for v in a]
    return (C.c_int32 * len(vals))(*vals)


def layout_check(N: int, Q: int, S: int, E: int, slot_expert, primary_slot=None) -> int:
    """Host-only validation of a layout; returns the status code (no device needed)."""
    se = _host_i32(slot_expert)
    if len(se) != N * Q * S:
        return ERR_INVALID_ARG
    pr = None if primary_slot is None else _host_i32(primary_slot)
    if pr is not None and len(pr) != E:
        return ERR_INVALID_ARG
    return _lib.cobalt_layout_check(N, Q, S, E, se, pr)


class Layout:
    """Owns a cobalt_layout_t (device tables of R_{e,n}, N_e and the primaries)."""

    def __init__(self, N: int, Q: int, S: int, E: int, slot_expert, primary_slot=None):
        se = _host_i32(slot_expert)
        if len(se) != N * Q * S:
            raise CobaltError(ERR_INVALID_ARG, "layout_create (slot_expert size)")
        pr = None if primary_slot is None else _host_i32(primary_slot)
        if pr is not None and len(pr) != E:
            raise CobaltError(ERR_INVALID_ARG, "layout_create (primary_slot size)")
        handle = C.c_void_p()
        _check(_lib.cobalt_layout_create(C.byref(handle), N, Q, S, E, se, pr), "cobalt_layout_create")
        self._h = handle
        self.N, self.Q, self.S, self.E = N, Q, S, E
        self.G, self.D = N * Q, N * Q * S

    @property
    def handle(self) -> C.c_void_p:
        if self._h is None:
            raise CobaltError(ERR_INVALID_ARG, "layout already destroyed")
        return self._h

    def destroy(self) -> None:
        if getattr(self, "_h", None) is not None:
            h, self._h = self._h, None
            _check(_lib.cobalt_layout_destroy(h), "cobalt_layout_destroy")

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def coact_stats_workspace_bytes(T: int, K: int, E: int) -> int:
    return _lib.cobalt_coact_stats_workspace_bytes(T, K, E)


def coact_stats(topk_ids: torch.Tensor, E: int, coact: torch.Tensor, load: torch.Tensor, *,
                flags: int = 0, workspace: Optional[torch.Tensor] = None) -> None:
    T, K = topk_ids.shape
    if coact.numel() != E * E or load.numel() != E:
        raise CobaltError(ERR_INVALID_ARG, "coact_stats (output sizes)")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.cobalt_coact_stats(_ptr(topk_ids, torch.int32, "topk_ids"), T, K, E,
                                   _ptr(coact, torch.int32, "coact"), _ptr(load, torch.int32, "load"), flags,
                                   _ptr(workspace), ws_bytes, _stream()), "cobalt_coact_stats")


def assign_workspace_bytes(layout: Layout, T: int, K: int) -> int:
    return _lib.cobalt_assign_workspace_bytes(layout.handle, T, K)


def assign(layout: Layout, topk_ids: torch.Tensor, src_rank, seed: int, assigned_slot: torch.Tensor, *,
           slot_load: Optional[torch.Tensor] = None, remote_nodes: Optional[torch.Tensor] = None,
           totals: Optional[torch.Tensor] = None, flags: int = 0,
           workspace: Optional[torch.Tensor] = None) -> None:
    """src_rank: int32 tensor [T], or a Python int used for every token.  seed: a Python int, or a
    one-element int64 CUDA tensor read when the kernel runs."""
    T, K = topk_ids.shape
    if assigned_slot.numel() != T * K:
        raise CobaltError(ERR_INVALID_ARG, "assign (assigned_slot size)")
    if slot_load is not None and slot_load.numel() != layout.D:
        raise CobaltError(ERR_INVALID_ARG, "assign (slot_load size)")
    if remote_nodes is not None and remote_nodes.numel() != T:
        raise CobaltError(ERR_INVALID_ARG, "assign (remote_nodes size)")
    if totals is not None and totals.numel() != 2:
        raise CobaltError(ERR_INVALID_ARG, "assign (totals size)")
    if isinstance(src_rank, int):
        src_ptr, src_uniform = None, src_rank
    else:
        if src_rank.numel() != T:
            raise CobaltError(ERR_INVALID_ARG, "assign (src_rank size)")
        src_ptr, src_uniform = _ptr(src_rank, torch.int32, "src_rank"), 0
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    seed, flags = _seed_arg(seed, flags)
    _check(_lib.cobalt_assign(layout.handle, _ptr(topk_ids, torch.int32, "topk_ids"), src_ptr, src_uniform,
                              T, K, seed, _ptr(assigned_slot, torch.int32, "assigned_slot"),
                              _ptr(slot_load, torch.int32, "slot_load"),
                              _ptr(remote_nodes, torch.uint8, "remote_nodes"),
                              _ptr(totals, torch.int64, "totals"), flags, _ptr(workspace), ws_bytes,
                              _stream()), "cobalt_assign")


def route_index_workspace_bytes(layout: Layout, T: int, K: int) -> int:
    return _lib.cobalt_route_index_workspace_bytes(layout.handle, T, K)


def route_index(layout: Layout, topk_ids: torch.Tensor, src_rank, seed: int, coact: torch.Tensor,
                load: torch.Tensor, assigned_slot: torch.Tensor, dest_counts: torch.Tensor,
                dest_offsets: torch.Tensor, row_of_pair: torch.Tensor, workspace: torch.Tensor, *,
                remote_nodes: Optional[torch.Tensor] = None, totals: Optional[torch.Tensor] = None,
                pair_of_row: Optional[torch.Tensor] = None, flags: int = 0) -> None:
    """Statistics, assignment and the permutation index in one pass over the ids."""
    T, K = topk_ids.shape
    E, D = layout.E, layout.D
    if coact.numel() != E * E or load.numel() != E or assigned_slot.numel() != T * K:
        raise CobaltError(ERR_INVALID_ARG, "route_index (output sizes)")
    _check_index_outputs(T, K, D, dest_counts, dest_offsets, row_of_pair, pair_of_row, "route_index")
    if remote_nodes is not None and remote_nodes.numel() != T:
        raise CobaltError(ERR_INVALID_ARG, "route_index (remote_nodes size)")
    if totals is not None and totals.numel() != 2:
        raise CobaltError(ERR_INVALID_ARG, "route_index (totals size)")
    if isinstance(src_rank, int):
        src_ptr, src_uniform = None, src_rank
    else:
        if src_rank.numel() != T:
            raise CobaltError(ERR_INVALID_ARG, "route_index (src_rank size)")
        src_ptr, src_uniform = _ptr(src_rank, torch.int32, "src_rank"), 0
    seed, flags = _seed_arg(seed, flags)
    _check(_lib.cobalt_route_index(layout.handle, _ptr(topk_ids, torch.int32, "topk_ids"), src_ptr, src_uniform, T, K,
                                   seed, _ptr(coact, torch.int32, "coact"),
                                   _ptr(load, torch.int32, "load"), _ptr(assigned_slot, torch.int32, "assigned_slot"),
                                   _ptr(remote_nodes, torch.uint8, "remote_nodes"), _ptr(totals, torch.int64, "totals"),
                                   _ptr(dest_counts, torch.int32, "dest_counts"),
                                   _ptr(dest_offsets, torch.int32, "dest_offsets"),
                                   _ptr(row_of_pair, torch.int32, "row_of_pair"),
                                   _ptr(pair_of_row, torch.int32, "pair_of_row"), flags, _ptr(workspace),
                                   _ws_bytes(workspace), _stream()), "cobalt_route_index")


def permute_workspace_bytes(T: int, K: int, D: int) -> int:
    return _lib.cobalt_permute_workspace_bytes(T, K, D)


def _ws_bytes(workspace: Optional[torch.Tensor]) -> int:
    return 0 if workspace is None else workspace.numel() * workspace.element_size()


def _check_index_outputs(T, K, D, dest_counts, dest_offsets, row_of_pair, pair_of_row, what):
    if dest_counts.numel() != D or dest_offsets.numel() != D + 1 or row_of_pair.numel() != T * K or (
            pair_of_row is not None and pair_of_row.numel() != T * K):
        raise CobaltError(ERR_INVALID_ARG, f"{what} (output sizes)")


def permute_index(assigned_slot: torch.Tensor, D: int, dest_counts: torch.Tensor, dest_offsets: torch.Tensor,
                  row_of_pair: torch.Tensor, pair_of_row: Optional[torch.Tensor],
                  workspace: torch.Tensor) -> None:
    T, K = assigned_slot.shape
    _check_index_outputs(T, K, D, dest_counts, dest_offsets, row_of_pair, pair_of_row, "permute_index")
    _check(_lib.cobalt_permute_index(_ptr(assigned_slot, torch.int32, "assigned_slot"), T, K, D,
                                     _ptr(dest_counts, torch.int32, "dest_counts"),
                                     _ptr(dest_offsets, torch.int32, "dest_offsets"),
                                     _ptr(row_of_pair, torch.int32, "row_of_pair"),
                                     _ptr(pair_of_row, torch.int32, "pair_of_row"),
                                     _ptr(workspace), _ws_bytes(workspace), _stream()), "cobalt_permute_index")


def permute_index_static(assigned_slot: torch.Tensor, D: int, dest_counts: torch.Tensor,
                         dest_offsets: torch.Tensor, row_of_pair: torch.Tensor,
                         pair_of_row: Optional[torch.Tensor]) -> None:
    """permute_index for callers that cannot hand over device scratch (a framework hot path that
    bans allocator calls, a plugin given only its inputs and outputs, a fully committed memory
    pool): the scratch is a fixed 4 MiB array inside the library.  Same outputs as
    permute_index; raises with ERR_SCRATCH_LIMIT when D * chunks exceeds STATIC_SCRATCH_WORDS.
    Calls share that array, so do not let two of them overlap on the GPU; make the first call
    on a device outside stream capture (it looks up the array's address)."""
    T, K = assigned_slot.shape
    _check_index_outputs(T, K, D, dest_counts, dest_offsets, row_of_pair, pair_of_row, "permute_index_static")
    _check(_lib.cobalt_permute_index_static(_ptr(assigned_slot, torch.int32, "assigned_slot"), T, K, D,
                                            _ptr(dest_counts, torch.int32, "dest_counts"),
                                            _ptr(dest_offsets, torch.int32, "dest_offsets"),
                                            _ptr(row_of_pair, torch.int32, "row_of_pair"),
                                            _ptr(pair_of_row, torch.int32, "pair_of_row"), _stream()),
           "cobalt_permute_index_static")


def permute_rows(x: torch.Tensor, row_of_pair: torch.Tensor, K: int, send: torch.Tensor, *, flags: int = 0) -> None:
    T, H = x.shape
    if row_of_pair.numel() != T * K or send.numel() != T * K * H:
        raise CobaltError(ERR_INVALID_ARG, "permute_rows (sizes)")
    _check(_lib.cobalt_permute_rows(_ptr(x, torch.bfloat16, "x"), _ptr(row_of_pair, torch.int32, "row_of_pair"),
                                    T, K, H, _ptr(send, torch.bfloat16, "send"), flags, _stream()),
           "cobalt_permute_rows")


def permute(assigned_slot: torch.Tensor, D: int, x: torch.Tensor, send: torch.Tensor, dest_counts: torch.Tensor,
            dest_offsets: torch.Tensor, row_of_pair: torch.Tensor, pair_of_row: Optional[torch.Tensor],
            workspace: torch.Tensor, *, flags: int = 0) -> None:
    T, K = assigned_slot.shape
    H = x.shape[1]
    if x.shape[0] != T or send.numel() != T * K * H:
        raise CobaltError(ERR_INVALID_ARG, "permute (x / send sizes)")
    _check_index_outputs(T, K, D, dest_counts, dest_offsets, row_of_pair, pair_of_row, "permute")
    _check(_lib.cobalt_permute(_ptr(assigned_slot, torch.int32, "assigned_slot"), T, K, D,
                               _ptr(x, torch.bfloat16, "x"), H, _ptr(send, torch.bfloat16, "send"),
                               _ptr(dest_counts, torch.int32, "dest_counts"),
                               _ptr(dest_offsets, torch.int32, "dest_offsets"),
                               _ptr(row_of_pair, torch.int32, "row_of_pair"),
                               _ptr(pair_of_row, torch.int32, "pair_of_row"), flags,
                               _ptr(workspace), _ws_bytes(workspace), _stream()), "cobalt_permute")


def combine(expert_out: torch.Tensor, row_of_pair: torch.Tensor, gate_w: torch.Tensor, y: torch.Tensor, *,
            flags: int = 0) -> None:
    T, K = gate_w.shape
    H = y.shape[1]
    if y.shape[0] != T or expert_out.numel() != T * K * H or row_of_pair.numel() != T * K:
        raise CobaltError(ERR_INVALID_ARG, "combine (sizes)")
    _check(_lib.cobalt_combine(_ptr(expert_out, torch.bfloat16, "expert_out"),
                               _ptr(row_of_pair, torch.int32, "row_of_pair"),
                               _ptr(gate_w, torch.float32, "gate_w"), T, K, H, _ptr(y, torch.bfloat16, "y"),
                               flags, _stream()), "cobalt_combine")


def _elem_ptr(t: torch.Tensor, offset_elems: int) -> int:
    return t.data_ptr() + offset_elems * t.element_size()


def permute_rows_block(x: torch.Tensor, row_of_pair_block: torch.Tensor, K: int, send: torch.Tensor, t0: int,
                       t1: int, *, flags: int = 0) -> None:
    """cobalt_permute_rows on tokens t0:t1 only (x and send are the whole buffers; row_of_pair_block
    holds the rows of pairs t0*K : t1*K, which index the whole send buffer)."""
    T, H = x.shape
    if not (0 <= t0 <= t1 <= T) or row_of_pair_block.numel() != (t1 - t0) * K or send.numel() != T * K * H:
        raise CobaltError(ERR_INVALID_ARG, "permute_rows_block (sizes)")
    _ptr(x, torch.bfloat16, "x"), _ptr(send, torch.bfloat16, "send")
    _check(_lib.cobalt_permute_rows_block(_elem_ptr(x, t0 * H), _ptr(row_of_pair_block, torch.int32, "row_of_pair"),
                                          t1 - t0, K, H, send.data_ptr(), T * K, flags, _stream()),
           "cobalt_permute_rows_block")


def combine_block(expert_out: torch.Tensor, row_of_pair_block: torch.Tensor, gate_w: torch.Tensor,
                  y: torch.Tensor, t0: int, t1: int, *, flags: int = 0) -> None:
    """cobalt_combine on tokens t0:t1 only (expert_out is the whole [P, H] buffer)."""
    T, K = gate_w.shape
    H = y.shape[1]
    if not (0 <= t0 <= t1 <= T) or row_of_pair_block.numel() != (t1 - t0) * K or expert_out.numel() != T * K * H:
        raise CobaltError(ERR_INVALID_ARG, "combine_block (sizes)")
    _ptr(expert_out, torch.bfloat16, "expert_out"), _ptr(gate_w, torch.float32, "gate_w"), _ptr(y, torch.bfloat16, "y")
    _check(_lib.cobalt_combine_block(expert_out.data_ptr(), _ptr(row_of_pair_block, torch.int32, "row_of_pair"),
                                     _elem_ptr(gate_w, t0 * K), t1 - t0, K, H, _elem_ptr(y, t0 * H), T * K, flags,
                                     _stream()), "cobalt_combine_block")


def permute_backward(grad_send: torch.Tensor, row_of_pair: torch.Tensor, K: int, grad_x: torch.Tensor, *,
                     flags: int = 0) -> None:
    """grad_x[t] = sum of the K rows of grad_send that token t was sent to."""
    T, H = grad_x.shape
    if row_of_pair.numel() != T * K or grad_send.numel() != T * K * H:
        raise CobaltError(ERR_INVALID_ARG, "permute_backward (sizes)")
    _check(_lib.cobalt_permute_backward(_ptr(grad_send, torch.bfloat16, "grad_send"),
                                        _ptr(row_of_pair, torch.int32, "row_of_pair"), T, K, H,
                                        _ptr(grad_x, torch.bfloat16, "grad_x"), flags, _stream()),
           "cobalt_permute_backward")


def combine_backward(grad_y: torch.Tensor, expert_out: Optional[torch.Tensor], row_of_pair: torch.Tensor,
                     gate_w: torch.Tensor, grad_expert_out: Optional[torch.Tensor],
                     grad_gate_w: Optional[torch.Tensor], *, flags: int = 0) -> None:
    T, K = gate_w.shape
    H = grad_y.shape[1]
    if grad_y.shape[0] != T or row_of_pair.numel() != T * K:
        raise CobaltError(ERR_INVALID_ARG, "combine_backward (sizes)")
    for name, t in (("expert_out", expert_out), ("grad_expert_out", grad_expert_out)):
        if t is not None and t.numel() != T * K * H:
            raise CobaltError(ERR_INVALID_ARG, f"combine_backward ({name} size)")
    if grad_gate_w is not None and grad_gate_w.numel() != T * K:
        raise CobaltError(ERR_INVALID_ARG, "combine_backward (grad_gate_w size)")
    _check(_lib.cobalt_combine_backward(_ptr(grad_y, torch.bfloat16, "grad_y"),
                                        _ptr(expert_out, torch.bfloat16, "expert_out"),
                                        _ptr(row_of_pair, torch.int32, "row_of_pair"),
                                        _ptr(gate_w, torch.float32, "gate_w"), T, K, H,
                                        _ptr(grad_expert_out, torch.bfloat16, "grad_expert_out"),
                                        _ptr(grad_gate_w, torch.float32, "grad_gate_w"), flags, _stream()),
           "cobalt_combine_backward")


def ema_update(counts: torch.Tensor, ema: torch.Tensor, decay: float, *, flags: int = 0) -> None:
    """ema = decay * ema + (1 - decay) * counts, element-wise on the device (counts int32, ema float32)."""
    if counts.numel() != ema.numel():
        raise CobaltError(ERR_INVALID_ARG, "ema_update (sizes)")
    _check(_lib.cobalt_ema_update(_ptr(counts, torch.int32, "counts"), _ptr(ema, torch.float32, "ema"),
                                  counts.numel(), decay, flags, _stream()), "cobalt_ema_update")


def ochiai(coact: torch.Tensor, out: torch.Tensor) -> None:
    E = coact.shape[0]
    if coact.numel() != E * E or out.numel() != E * E:
        raise CobaltError(ERR_INVALID_ARG, "ochiai (sizes)")
    _check(_lib.cobalt_ochiai(_ptr(coact, torch.int32, "coact"), E, _ptr(out, torch.float32, "ochiai"), _stream()),
           "cobalt_ochiai")


def rebalance_intra_node(N: int, Q: int, S: int, E: int, slot_expert, slot_load):
    """Stage-2 greedy rebalancing on host arrays -> (new_slot_expert, moved_from, nodes_kept) as Python lists/int."""
    D = N * Q * S
    se = _host_i32(slot_expert)
    ld = (C.c_float * D)(*[float(v) for v in slot_load])
    if len(se) != D:
        raise CobaltError(ERR_INVALID_ARG, "rebalance_intra_node (slot_expert size)")
    new = (C.c_int32 * D)()
    moved = (C.c_int32 * D)()
    kept = C.c_int32(0)
    _check(_lib.cobalt_rebalance_intra_node(N, Q, S, E, se, ld, new, moved, C.byref(kept)),
           "cobalt_rebalance_intra_node")
    return list(new), list(moved), int(kept.value)


def dedup_workspace_bytes(T: int, K: int, N: int) -> int:
    return _lib.cobalt_dedup_workspace_bytes(T, K, N)


def dedup_index(assigned_slot: torch.Tensor, src_rank, N: int, Q: int, S: int, node_counts: torch.Tensor,
                node_offsets: torch.Tensor, node_row_of_token: torch.Tensor, fwd_src_row: torch.Tensor,
                workspace: torch.Tensor, *, cross_node_rows: Optional[torch.Tensor] = None) -> None:
    """One row per (token, destination node): see cobalt_dedup_index."""
    T, K = assigned_slot.shape
    if (node_counts.numel() != N or node_offsets.numel() != N + 1 or node_row_of_token.numel() != T * N or
            fwd_src_row.numel() != T * K or (cross_node_rows is not None and cross_node_rows.numel() != 1)):
        raise CobaltError(ERR_INVALID_ARG, "dedup_index (output sizes)")
    if isinstance(src_rank, int):
        src_ptr, src_uniform = None, src_rank
    else:
        src_ptr, src_uniform = _ptr(src_rank, torch.int32, "src_rank"), 0
    _check(_lib.cobalt_dedup_index(_ptr(assigned_slot, torch.int32, "assigned_slot"), src_ptr, src_uniform, T, K,
                                   N, Q, S, _ptr(node_counts, torch.int32, "node_counts"),
                                   _ptr(node_offsets, torch.int32, "node_offsets"),
                                   _ptr(node_row_of_token, torch.int32, "node_row_of_token"),
                                   _ptr(fwd_src_row, torch.int32, "fwd_src_row"),
                                   _ptr(cross_node_rows, torch.int64, "cross_node_rows"), _ptr(workspace),
                                   _ws_bytes(workspace), _stream()), "cobalt_dedup_index")


def dedup_rows(x: torch.Tensor, node_row_of_token: torch.Tensor, N: int, dedup_send: torch.Tensor, *,
               flags: int = 0) -> None:
    """Fill the deduplicated buffer: the row mover with N optional copies per token."""
    T, H = x.shape
    if node_row_of_token.numel() != T * N or dedup_send.shape[1] != H:
        raise CobaltError(ERR_INVALID_ARG, "dedup_rows (sizes)")
    _check(_lib.cobalt_permute_rows_block(_ptr(x, torch.bfloat16, "x"),
                                          _ptr(node_row_of_token, torch.int32, "node_row_of_token"), T, N, H,
                                          _ptr(dedup_send, torch.bfloat16, "dedup_send"), dedup_send.shape[0], flags,
                                          _stream()), "cobalt_permute_rows_block")


def forward_rows(dedup_send: torch.Tensor, fwd_src_row: torch.Tensor, row_of_pair: torch.Tensor,
                 recv: torch.Tensor) -> None:
    """recv[row_of_pair[p]] = dedup_send[fwd_src_row[p]]."""
    P = fwd_src_row.numel()
    H = dedup_send.shape[1]
    if row_of_pair.numel() != P or recv.shape[1] != H:
        raise CobaltError(ERR_INVALID_ARG, "forward_rows (sizes)")
    _check(_lib.cobalt_forward_rows(_ptr(dedup_send, torch.bfloat16, "dedup_send"),
                                    _ptr(fwd_src_row, torch.int32, "fwd_src_row"),
                                    _ptr(row_of_pair, torch.int32, "row_of_pair"), P, H,
                                    _ptr(recv, torch.bfloat16, "recv"), dedup_send.shape[0], recv.shape[0], _stream()),
           "cobalt_forward_rows")


def read_and_clear_device_error() -> int:
    bits = C.c_uint32(0)
    _check(_lib.cobalt_read_and_clear_device_error(C.byref(bits), _stream()),
           "cobalt_read_and_clear_device_error")
    return int(bits.value)
