"""The C oracle and the library's host-only code under AddressSanitizer and UndefinedBehaviorSanitizer.

compute-sanitizer is not available for the device code, so the host side at least is run
instrumented: a plain C driver walks the oracle through the Fig. 1 example, a ragged eight-node
case and the inputs it must refuse; a second one walks the library's layout validation and Stage-2
rebalancer (runtime.cu and epilogue.cu built with the sanitizers on their host code).  Any report
aborts the driver (-fno-sanitize-recover), which fails the test.
"""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SAN = ["-fsanitize=address", "-fsanitize=undefined", "-fno-sanitize-recover=all"]
ENV = dict(os.environ, ASAN_OPTIONS="detect_leaks=1:protect_shadow_gap=0:abort_on_error=0",
           UBSAN_OPTIONS="print_stacktrace=1")


def run(cmd, **kw):
    r = subprocess.run(cmd, capture_output=True, text=True, **kw)
    assert r.returncode == 0, " ".join(cmd) + "\n" + r.stdout + r.stderr
    return r.stdout


def test_oracle_under_sanitizers(tmp_path):
    exe = str(tmp_path / "oracle_check")
    run(["gcc", "-std=c11", "-O1", "-g", "-Wall", "-Wextra", *SAN, "-ffp-contract=off",
         os.path.join(ROOT, "oracle", "cobalt_oracle.c"), os.path.join(ROOT, "tests", "sanitize", "oracle_check.c"),
         "-o", exe])
    assert "oracle ok under the sanitizers" in run([exe], env=ENV)


@pytest.mark.skipif(shutil.which(os.environ.get("NVCC", "nvcc")) is None, reason="nvcc builds the .cu host code")
def test_library_host_code_under_sanitizers(tmp_path):
    nvcc = os.environ.get("NVCC", "nvcc")
    csrc = os.path.join(ROOT, "paper_2609_36959_b200", "csrc")
    obj, exe = str(tmp_path / "host_check.o"), str(tmp_path / "host_check")
    run(["gcc", "-std=c11", "-O1", "-g", "-Wall", "-Wextra", *SAN, "-I", os.path.join(ROOT, "include"), "-c",
         os.path.join(ROOT, "tests", "sanitize", "host_check.c"), "-o", obj])
    xc = [a for flag in SAN for a in ("-Xcompiler", flag)]
    run([nvcc, "-O1", "-g", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", *xc,
         "-I", os.path.join(ROOT, "include"), "-I", csrc, os.path.join(csrc, "runtime.cu"),
         os.path.join(csrc, "epilogue.cu"), obj, "-o", exe])
    # the CUDA runtime's own start-up allocations are not this library's: leak checking off here
    env = dict(ENV, ASAN_OPTIONS="detect_leaks=0:protect_shadow_gap=0")
    assert "host entry points ok under the sanitizers" in run([exe], env=env)
