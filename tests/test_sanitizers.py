"""AddressSanitizer + UndefinedBehaviorSanitizer over the host code (no GPU needed).

tests/sanitize_driver.c is compiled with the sanitizers together with the oracle's C source and run on ordinary and
degenerate inputs; then the same driver, still under the sanitizers, loads a copy of libpolyspec.so whose HOST code was
compiled with the sanitizers as well and calls the C ABI's size queries and argument checks with bad arguments -- the
paths that must return a status before any CUDA call.  A finding aborts the driver with a report.
"""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SAN = ["-fsanitize=address,undefined", "-fno-sanitize-recover=undefined", "-fno-omit-frame-pointer", "-g"]
ENV = dict(os.environ, ASAN_OPTIONS="detect_leaks=1:abort_on_error=0:protect_shadow_gap=0", UBSAN_OPTIONS="print_stacktrace=1")


def _driver(tmp_path):
    exe = str(tmp_path / "sanitize_driver")
    cmd = ["gcc", "-O1", "-std=c99", *SAN, "-o", exe, os.path.join(ROOT, "tests", "sanitize_driver.c"),
           os.path.join(ROOT, "oracle", "polyspec_oracle.c"), "-lm", "-ldl"]
    subprocess.run(cmd, check=True, capture_output=True, text=True)
    return exe


def test_oracle_under_address_and_undefined_behaviour_sanitizers(tmp_path):
    exe = _driver(tmp_path)
    res = subprocess.run([exe], capture_output=True, text=True, env=ENV, timeout=300)
    assert res.returncode == 0, res.stdout + res.stderr
    assert "0 failed checks" in res.stdout


def test_abi_argument_checks_under_sanitizers(tmp_path):
    from paper_2510_26527_b200 import buildlib
    nvcc = buildlib._nvcc()
    lib = str(tmp_path / "libpolyspec_san.so")
    host = []
    for f in ("-fsanitize=address", "-fsanitize=undefined", "-fno-sanitize-recover=undefined", "-fno-omit-frame-pointer"):
        host += ["-Xcompiler", f]
    cmd = [nvcc, *buildlib.NVCC_FLAGS, *host, "-I", buildlib.INCLUDE, "-I", buildlib.CSRC, "-o", lib, *buildlib.sources()]
    res = subprocess.run(cmd, capture_output=True, text=True)
    assert res.returncode == 0, res.stdout + res.stderr
    exe = _driver(tmp_path)
    res = subprocess.run([exe, lib], capture_output=True, text=True, env=ENV, timeout=300)
    assert res.returncode == 0, res.stdout + res.stderr
    assert "0 failed checks" in res.stdout
