"""CPU-only checks of the C-ABI boundary: the library loads, exports every declared symbol,
and its host-side logic (status strings, layout validation, workspace sizing, argument checks
that run before any device work) behaves as documented.  No kernel is launched here."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    from paper_2609_36959_b200 import build
    return build.build()


@pytest.fixture(scope="module")
def cb(lib_path):
    import paper_2609_36959_b200.binding as binding
    return binding


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "cobalt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cobalt_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib_path, cb):
    lib = C.CDLL(lib_path)
    names = declared_symbols()
    assert len(names) >= 17
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in cobalt.h but not exported"
    assert sorted(cb.EXPORTS) == names


def test_library_exports_nothing_beyond_the_header(lib_path):
    """The dynamic symbol table lists exactly the header's cobalt_* functions: no tuning hooks or
    other undeclared entry points ship in the library."""
    import subprocess
    out = subprocess.run(["nm", "-D", "--defined-only", lib_path], capture_output=True, text=True, check=True).stdout
    exported = sorted({line.split()[-1] for line in out.splitlines()
                       if line.split() and line.split()[-1].startswith("cobalt_") and " T " in line})
    assert exported == declared_symbols()


def test_measurement_library_exports_its_header():
    """libcobalt_peaks.so (the benchmark's measurement kernels) exports exactly what cobalt_peaks.h declares."""
    import subprocess
    from paper_2609_36959_b200 import build, peaks
    lib = build.build_peaks()
    with open(os.path.join(ROOT, "include", "cobalt_peaks.h")) as f:
        declared = sorted(set(re.findall(r"\b(cobalt_[a-z_0-9]+)\s*\(", f.read())))
    out = subprocess.run(["nm", "-D", "--defined-only", lib], capture_output=True, text=True, check=True).stdout
    exported = sorted({line.split()[-1] for line in out.splitlines()
                       if line.split() and line.split()[-1].startswith("cobalt_") and " T " in line})
    assert exported == declared == sorted(peaks.EXPORTS)


def test_version_and_status_strings(cb):
    assert cb.version() == 100
    seen = {cb.status_string(s) for s in (0, -1, -2, -3, -4, -5, -6)}
    assert len(seen) == 7 and "unknown status" not in seen
    assert cb.status_string(-99) == "unknown status"


def test_layout_check_accepts_fig1_and_rejects_bad_layouts(cb, fig1):
    g = fig1
    assert cb.layout_check(2, 2, 2, 4, g["slot_expert"], g["primary_slot"]) == cb.OK
    assert cb.layout_check(2, 2, 2, 4, g["slot_expert"], None) == cb.OK
    assert cb.layout_check(2, 2, 2, 4, [0, -1, 1, -1, 2, -1, 3, 0]) == cb.OK              # empty slots
    assert cb.layout_check(2, 2, 2, 4, [0, 1, 2, 0, 1, 2, 0, 0]) == cb.ERR_INVALID_ARG     # expert 3 missing
    assert cb.layout_check(2, 2, 2, 4, [0, 0, 2, 1, 1, 2, 3, 0]) == cb.ERR_INVALID_ARG     # twice on a rank
    assert cb.layout_check(2, 2, 2, 4, [0, 1, 2, 0, 1, 2, 3, 4]) == cb.ERR_INVALID_ARG     # id out of range
    assert cb.layout_check(2, 2, 2, 4, g["slot_expert"], [1, 4, 2, 6]) == cb.ERR_INVALID_ARG
    assert cb.layout_check(2, 2, 2, 4, g["slot_expert"][:-1]) == cb.ERR_INVALID_ARG
    assert cb.layout_check(9, 1, 1, 9, list(range(9))) == cb.ERR_UNSUPPORTED               # N > 8
    assert cb.layout_check(0, 2, 2, 4, []) == cb.ERR_INVALID_ARG


def test_layout_check_agrees_with_the_oracle_on_generated_layouts(cb):
    import oracle as O
    import workloads as W
    for name in W.CONFIG_NAMES:
        w = W.make_config(name, T=16)
        assert cb.layout_check(w.N, w.Q, w.S, w.E, w.slot_expert.tolist(), w.primary_slot.tolist()) == cb.OK
        O.layout_tables(w.N, w.Q, w.S, w.E, w.slot_expert, w.primary_slot)


def test_workspace_queries(cb):
    assert cb.coact_stats_workspace_bytes(131072, 8, 256) == 0
    small = cb.permute_workspace_bytes(4096, 2, 24)
    big = cb.permute_workspace_bytes(131072, 8, 288)
    assert small > 0 and big >= 288 * 512 * 4 and big % 256 == 0
    assert cb.permute_workspace_bytes(10, 2, 5000) == 0          # D outside the envelope


def test_argument_checks_run_before_any_device_work(cb):
    lib = cb._lib
    # NULL outputs / negative sizes / unsupported shapes are refused without touching CUDA
    assert lib.cobalt_coact_stats(None, 16, 2, 8, None, None, 0, None, 0, None) == cb.ERR_INVALID_ARG
    assert lib.cobalt_coact_stats(None, -1, 2, 8, 16, 16, 0, None, 0, None) == cb.ERR_INVALID_ARG
    assert lib.cobalt_coact_stats(None, 16, 17, 32, 16, 16, 0, None, 0, None) == cb.ERR_UNSUPPORTED
    assert lib.cobalt_assign(None, None, None, 0, 16, 2, 1, None, None, None, None, 0, None, 0, None) == cb.ERR_INVALID_ARG
    assert lib.cobalt_permute_index(16, 4, 2, 8, None, None, 16, None, None, 0, None) == cb.ERR_INVALID_ARG
    assert lib.cobalt_permute_index(16, 4, 2, 5000, 16, 16, 16, None, None, 0, None) == cb.ERR_UNSUPPORTED
    assert lib.cobalt_permute_index(16, 4, 2, 8, 16, 16, 16, None, None, 0, None) == cb.ERR_WORKSPACE_TOO_SMALL
    assert lib.cobalt_permute_rows(16, 16, 4, 2, 12, 16, 0, None) == cb.ERR_UNSUPPORTED      # H % 8 != 0
    assert lib.cobalt_permute_rows(8, 16, 4, 2, 16, 16, 0, None) == cb.ERR_INVALID_ARG       # misaligned x
    assert lib.cobalt_combine(16, 16, 16, 4, 2, 16, None, 0, None) == cb.ERR_INVALID_ARG
    assert lib.cobalt_combine(16, 16, 16, 4, 17, 16, 16, 0, None) == cb.ERR_UNSUPPORTED
    assert lib.cobalt_read_and_clear_device_error(None, None) == cb.ERR_INVALID_ARG


def test_binding_refuses_host_tensors(cb):
    import torch
    ids = torch.zeros((4, 2), dtype=torch.int32)
    out = torch.zeros((8, 8), dtype=torch.int32)
    with pytest.raises(TypeError):
        cb.coact_stats(ids, 8, out, out[0])


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    """No fallback: importing the binding without the shared library raises."""
    import importlib
    import paper_2609_36959_b200.binding as binding
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "libcobalt.so"))
    with pytest.raises(ImportError):
        binding._load()
    importlib.reload(binding)
