"""The C-ABI library on a machine without a GPU: it loads, exports every symbol the header declares,
answers the host-only calls, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2510_26527_b200 import binding, buildlib

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    buildlib.build()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "polyspec.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(polyspec_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_version_and_status_strings(lib):
    assert binding.version() >= 100
    seen = {binding.status_string(s) for s in range(7)}
    assert len(seen) == 7 and "ok" in seen
    assert binding.status_string(99) == "unknown status"


def test_workspace_queries_are_host_only(lib):
    n1 = binding.polyspec_verify_level_workspace(1, 4, 32000, binding.F32)
    n5 = binding.polyspec_verify_chain_workspace([4, 6, 10], [5, 7, 11, 10], 256, 152064, binding.BF16)
    assert n1 % 256 == 0 and n1 >= 9 * 8
    assert n5 % 256 == 0 and n5 >= 8448 * 8
    nh = binding.polyspec_verify_chain_host_workspace([4, 6, 10], [5, 7, 11, 10], 256, 152064, binding.BF16)
    assert nh > 256 * 33 * 152064 * 2                  # holds a staged copy of every logits row
    nf = binding.polyspec_verify_from_hidden_workspace(32, 8, 32000, 4096, 2048)
    assert nf > 2 * 288 * 32000 * 4


@pytest.mark.parametrize("args,status", [
    ((0, 4, 32000, binding.F32), binding.ERR_INVALID_ARG),          # B <= 0
    ((1, 0, 32000, binding.F32), binding.ERR_INVALID_ARG),          # k < 1
    ((1, 33, 32000, binding.F32), binding.ERR_INVALID_ARG),         # k > POLYSPEC_MAX_K
    ((1, 4, 32001, binding.F32), binding.ERR_UNSUPPORTED),          # V not a multiple of 8
    ((1, 4, 32000, 7), binding.ERR_INVALID_ARG),                    # unknown dtype
])
def test_workspace_query_rejects_bad_sizes(lib, args, status):
    n = ctypes.c_size_t(0)
    assert lib.polyspec_verify_level_workspace(*args, ctypes.byref(n)) == status


def test_calls_reject_bad_arguments_without_launching(lib):
    # NULL pointers, a bad temperature and a short workspace are caught on the host: no CUDA call is made
    null = None
    st = lib.polyspec_verify_level(null, null, null, null, null, 1, 4, 32000, binding.F32, 1.0,
                                   null, null, null, null, null, null, 0, null)
    assert st == binding.ERR_INVALID_ARG
    fake = 0x1000                                       # aligned, never dereferenced on the host
    for temp in (0.0, -1.0, float("nan"), float("inf")):
        st = lib.polyspec_verify_level(fake, fake, fake, fake, null, 1, 4, 32000, binding.F32, temp,
                                       fake, fake, null, null, null, fake, 1 << 20, null)
        assert st == binding.ERR_INVALID_ARG
    st = lib.polyspec_verify_level(fake, fake, fake, fake, null, 1, 4, 32000, binding.F32, 1.0,
                                   fake, fake, null, null, null, fake, 8, null)
    assert st == binding.ERR_WORKSPACE
    st = lib.polyspec_verify_level(fake + 4, fake, fake, fake, null, 1, 4, 32000, binding.F32, 1.0,
                                   fake, fake, null, null, null, fake, 1 << 20, null)
    assert st == binding.ERR_INVALID_ARG                # logits not 16-byte aligned
    k = (ctypes.c_int * 2)(9, 8)
    models = (binding.ModelLogits * 3)(binding.ModelLogits(fake, 10), binding.ModelLogits(fake, 8), binding.ModelLogits(fake, 8))
    st = lib.polyspec_verify_chain(models, 3, k, fake, fake, 1, 32000, binding.BF16, 1.0,
                                   fake, fake, fake, fake, null, fake, 1 << 20, null)
    assert st == binding.ERR_INVALID_ARG                # model 1 has fewer rows than k[1] + 1
    st = lib.polyspec_verify_from_hidden(fake, fake, fake, fake, 9, fake, fake, null, 32, 8, 32000, 4096, 2050, 1.0,
                                         fake, fake, null, null, null, fake, 1 << 30, null)
    assert st == binding.ERR_UNSUPPORTED                # d_q not a multiple of 64


def test_binding_raises_when_the_library_is_missing(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libpolyspec.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load_library()
