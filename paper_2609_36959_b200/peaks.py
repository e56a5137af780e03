"""ctypes binding of libcobalt_peaks.so: the measurement kernels behind the benchmark's second
roofline (shared-memory atomic adds and warp instructions per clock and SM).  Not part of the
routing path; see include/cobalt_peaks.h."""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libcobalt_peaks.so")

EXPORTS = ("cobalt_peak_shared_atomics", "cobalt_peak_issue_rate")


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_36959_b200.build`")
    lib = C.CDLL(LIB_PATH)
    lib.cobalt_peak_shared_atomics.restype = C.c_int
    lib.cobalt_peak_shared_atomics.argtypes = [C.c_int, C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_int32,
                                               C.POINTER(C.c_double)]
    lib.cobalt_peak_issue_rate.restype = C.c_int
    lib.cobalt_peak_issue_rate.argtypes = [C.c_int32, C.c_int32, C.POINTER(C.c_double)]
    return lib


_lib = _load()


def shared_atomics_conflict_free(repeats: int = 64) -> float:
    """Shared-memory atomic adds per clock and SM when no two lanes of a warp share a bank."""
    out = C.c_double(0.0)
    rc = _lib.cobalt_peak_shared_atomics(0, None, 0, 0, 0, repeats, C.byref(out))
    if rc != 0:
        raise RuntimeError(f"cobalt_peak_shared_atomics: cuda error {rc}")
    return out.value


def shared_atomics_stats_pattern(topk_ids: torch.Tensor, E: int, repeats: int = 8) -> float:
    """The same rate for the statistics stage's own adds over these tokens (int32 [T, K] on the device)."""
    if not topk_ids.is_cuda or topk_ids.dtype != torch.int32 or not topk_ids.is_contiguous():
        raise TypeError("topk_ids must be a contiguous int32 CUDA tensor")
    T, K = topk_ids.shape
    out = C.c_double(0.0)
    rc = _lib.cobalt_peak_shared_atomics(1, topk_ids.data_ptr(), T, K, E, repeats, C.byref(out))
    if rc != 0:
        raise RuntimeError(f"cobalt_peak_shared_atomics: cuda error {rc}")
    return out.value


def issue_rate(mix: int = 0, repeats: int = 64) -> float:
    """Warp instructions per clock and SM of 32 resident warps running independent integer arithmetic
    (mix 0: add/shift/logic, mix 1: the multiply-add/shift/logic mix of the counter hash)."""
    out = C.c_double(0.0)
    rc = _lib.cobalt_peak_issue_rate(mix, repeats, C.byref(out))
    if rc != 0:
        raise RuntimeError(f"cobalt_peak_issue_rate: cuda error {rc}")
    return out.value
