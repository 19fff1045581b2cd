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


def test_greedy_fused_and_projection_calls_reject_bad_arguments_without_launching(lib):
    null = None
    fake = 0x1000
    k = (ctypes.c_int * 2)(4, 6)
    rows = (ctypes.c_int * 3)(5, 7, 6)
    n = ctypes.c_size_t(0)
    assert lib.polyspec_verify_chain_greedy_workspace(3, k, rows, 8, 32000, binding.BF16, ctypes.byref(n)) == binding.OK
    assert n.value % 256 == 0 and n.value > 0
    assert lib.polyspec_verify_chain_greedy_workspace(3, k, rows, 8, 32000, binding.BF16, null) == binding.ERR_INVALID_ARG
    assert lib.polyspec_verify_chain_greedy_workspace(1, k, rows, 8, 32000, binding.BF16, ctypes.byref(n)) == binding.ERR_INVALID_ARG
    assert lib.polyspec_verify_chain_greedy_workspace(3, k, rows, 8, 32004, binding.BF16, ctypes.byref(n)) == binding.ERR_UNSUPPORTED
    models = (binding.ModelLogits * 3)(binding.ModelLogits(fake, 5), binding.ModelLogits(fake, 7), binding.ModelLogits(null, 6))
    # the drafter's logits may be NULL under greedy matching; a verifier's may not
    st = lib.polyspec_verify_chain_greedy(models, 3, k, fake, 8, 32000, binding.BF16, fake, fake, fake, fake, null, fake, 8, null)
    assert st == binding.ERR_WORKSPACE
    models[1].logits = null
    st = lib.polyspec_verify_chain_greedy(models, 3, k, fake, 8, 32000, binding.BF16, fake, fake, fake, fake, null, fake, 1 << 30, null)
    assert st == binding.ERR_INVALID_ARG
    models[1].logits = fake
    st = lib.polyspec_verify_chain_greedy(models, 3, k, null, 8, 32000, binding.BF16, fake, fake, fake, fake, null, fake, 1 << 30, null)
    assert st == binding.ERR_INVALID_ARG                # no draft tokens
    st = lib.polyspec_verify_chain_greedy(models, 3, k, fake, 8, 32000, binding.BF16, fake, fake, fake, fake, null, fake + 16, 1 << 30, null)
    assert st == binding.ERR_INVALID_ARG                # workspace not 256-byte aligned

    # the projection alone
    assert lib.polyspec_lm_head(null, fake, 8, 32000, 4096, fake, null, null) == binding.ERR_INVALID_ARG
    assert lib.polyspec_lm_head(fake, fake, 0, 32000, 4096, fake, null, null) == binding.ERR_INVALID_ARG
    assert lib.polyspec_lm_head(fake + 8, fake, 8, 32000, 4096, fake, null, null) == binding.ERR_INVALID_ARG
    assert lib.polyspec_lm_head(fake, fake, 8, 32000, 4100, fake, null, null) == binding.ERR_UNSUPPORTED
    assert lib.polyspec_lm_head(fake, fake, 8, 32002, 4096, fake, null, null) == binding.ERR_UNSUPPORTED

    # the fused call and its halves
    f32 = ctypes.c_float
    args = dict(B=32, k=8, V=32000, dp=4096, dq=2048)
    assert lib.polyspec_verify_from_hidden_workspace(32, 8, 32000, 4096, 2048, ctypes.byref(n)) == binding.OK
    need = n.value

    def fused(rows_q=9, temp=1.0, ws=fake, ws_bytes=1 << 40, hp=fake, tokens=fake, nxt=fake, **kw):
        a = dict(args, **kw)
        return lib.polyspec_verify_from_hidden(hp, fake, fake, fake, rows_q, tokens, fake, null, a["B"], a["k"], a["V"], a["dp"], a["dq"],
                                               f32(temp), fake, nxt, null, null, null, ws, ws_bytes, null)
    assert fused(ws_bytes=need - 256) == binding.ERR_WORKSPACE
    assert fused(rows_q=7) == binding.ERR_INVALID_ARG       # fewer drafter rows than the block
    assert fused(rows_q=10) == binding.ERR_INVALID_ARG      # more than k + 1
    assert fused(temp=0.0) == binding.ERR_INVALID_ARG
    assert fused(hp=null) == binding.ERR_INVALID_ARG
    assert fused(tokens=null) == binding.ERR_INVALID_ARG
    assert fused(nxt=null) == binding.ERR_INVALID_ARG
    assert fused(ws=null) == binding.ERR_INVALID_ARG
    assert fused(k=33) == binding.ERR_INVALID_ARG
    assert fused(V=32004) == binding.ERR_UNSUPPORTED
    assert fused(dp=4100) == binding.ERR_UNSUPPORTED
    st = lib.polyspec_from_hidden_project(fake, fake, fake, fake, 9, 32, 8, 32000, 4096, 2048, f32(float("nan")), null, fake, 1 << 40, null)
    assert st == binding.ERR_INVALID_ARG
    st = lib.polyspec_from_hidden_verify(9, fake, null, null, 32, 8, 32000, 4096, 2048, f32(1.0), fake, fake, null, null, null,
                                         fake, 1 << 40, null)
    assert st == binding.ERR_INVALID_ARG                # no uniforms

    # the host-buffer chain call
    hk = (ctypes.c_int * 1)(4)
    hrows = (ctypes.c_int * 2)(5, 4)
    assert lib.polyspec_verify_chain_host_workspace(2, hk, hrows, 4, 32000, binding.F32, ctypes.byref(n)) == binding.OK
    hm = (binding.ModelLogits * 2)(binding.ModelLogits(fake, 5), binding.ModelLogits(fake, 4))
    st = lib.polyspec_verify_chain_host(hm, 2, hk, fake, fake, 4, 32000, binding.F32, f32(1.0), fake, fake, fake, fake, null,
                                        fake, n.value - 256, null)
    assert st == binding.ERR_WORKSPACE
    st = lib.polyspec_verify_chain_host(hm, 2, hk, null, fake, 4, 32000, binding.F32, f32(1.0), fake, fake, fake, fake, null,
                                        fake, n.value, null)
    assert st == binding.ERR_INVALID_ARG


def test_sharded_level_calls_reject_bad_arguments_without_launching(lib):
    null, fake = None, 0x1000
    f32 = ctypes.c_float
    w, a, m = ctypes.c_size_t(0), ctypes.c_size_t(0), ctypes.c_size_t(0)
    ok = lib.polyspec_sharded_level_sizes(64, 6, 16032, binding.BF16, 8, ctypes.byref(w), ctypes.byref(a), ctypes.byref(m))
    assert ok == binding.OK
    assert w.value % 256 == 0 and a.value >= 64 * (13 * 12 + 12 * 4) and m.value >= 64 * 16
    for args, st in (((0, 6, 16032, binding.BF16, 8), binding.ERR_INVALID_ARG),
                     ((64, 33, 16032, binding.BF16, 8), binding.ERR_INVALID_ARG),
                     ((64, 6, 16032, binding.BF16, 0), binding.ERR_INVALID_ARG),
                     ((64, 6, 16032, binding.BF16, 65), binding.ERR_INVALID_ARG),
                     ((64, 6, 16036, binding.BF16, 8), binding.ERR_UNSUPPORTED),        # slice not a multiple of 8
                     ((64, 6, 1 << 21, binding.BF16, 2048 // 64 * 64), binding.ERR_INVALID_ARG)):
        assert lib.polyspec_sharded_level_sizes(*args, ctypes.byref(w), ctypes.byref(a), ctypes.byref(m)) == st, args
    assert lib.polyspec_sharded_level_sizes(64, 6, 16032, binding.BF16, 8, null, ctypes.byref(a), ctypes.byref(m)) == binding.ERR_INVALID_ARG
    lib.polyspec_sharded_level_sizes(64, 6, 16032, binding.BF16, 8, ctypes.byref(w), ctypes.byref(a), ctypes.byref(m))

    def stats(rank=0, ws_bytes=1 << 40, rec=fake, temp=1.0, lp=fake):
        return lib.polyspec_sharded_level_stats(lp, fake, fake, 64, 6, 16032, rank, 8, binding.BF16, f32(temp), rec, null, fake, ws_bytes, null)
    assert stats(rank=8) == binding.ERR_INVALID_ARG
    assert stats(rank=-1) == binding.ERR_INVALID_ARG
    assert stats(ws_bytes=w.value - 256) == binding.ERR_WORKSPACE
    assert stats(rec=null) == binding.ERR_INVALID_ARG
    assert stats(temp=0.0) == binding.ERR_INVALID_ARG
    assert stats(lp=fake + 8) == binding.ERR_INVALID_ARG
    st = lib.polyspec_sharded_level_decide(fake, fake, fake, fake, null, 64, 6, 16032, 0, 8, binding.BF16, f32(1.0), null,
                                           fake, null, null, fake, null, fake, 1 << 40, null)
    assert st == binding.ERR_INVALID_ARG                # no stats records
    st = lib.polyspec_sharded_level_pick(fake, fake, fake, 64, 6, 16032, 0, 8, binding.BF16, f32(1.0), fake, null, null, fake, 1 << 40, null)
    assert st == binding.ERR_INVALID_ARG                # nowhere to put the token


def test_sharded_chain_calls_reject_bad_arguments_without_launching(lib):
    null, fake = None, 0x1000
    f32 = ctypes.c_float
    k = (ctypes.c_int * 3)(4, 6, 10)
    rows = (ctypes.c_int * 4)(5, 7, 11, 10)
    sizes = [ctypes.c_size_t(0) for _ in range(4)]
    refs = [ctypes.byref(x) for x in sizes]
    assert lib.polyspec_sharded_chain_sizes(4, k, rows, 256, 19008, binding.BF16, 8, *refs) == binding.OK
    w, a, g, m = (x.value for x in sizes)
    assert a >= 256 * 33 * 12 and g >= 256 * 11 * 8 and m >= 256 * 16 and all(x % 256 == 0 for x in (w, a, g, m))
    assert lib.polyspec_sharded_chain_sizes(1, k, rows, 256, 19008, binding.BF16, 8, *refs) == binding.ERR_INVALID_ARG
    assert lib.polyspec_sharded_chain_sizes(4, k, rows, 256, 19004, binding.BF16, 8, *refs) == binding.ERR_UNSUPPORTED
    short = (ctypes.c_int * 4)(5, 6, 11, 10)                           # model 1 lacks its bonus row
    assert lib.polyspec_sharded_chain_sizes(4, k, short, 256, 19008, binding.BF16, 8, *refs) == binding.ERR_INVALID_ARG
    models = (binding.ModelLogits * 4)(*[binding.ModelLogits(fake, r) for r in (5, 7, 11, 10)])
    st = lib.polyspec_sharded_chain_stats(models, 4, k, 256, 19008, 8, 8, binding.BF16, f32(1.0), fake, null, fake, 1 << 40, null)
    assert st == binding.ERR_INVALID_ARG                # rank out of range
    st = lib.polyspec_sharded_chain_stats(models, 4, k, 256, 19008, 0, 8, binding.BF16, f32(1.0), fake, null, fake, w - 256, null)
    assert st == binding.ERR_WORKSPACE
    st = lib.polyspec_sharded_chain_gather(models, 4, k, 3, fake, fake, 256, 19008, 0, 8, binding.BF16, fake, fake, 1 << 40, null)
    assert st == binding.ERR_INVALID_ARG                # no such level
    st = lib.polyspec_sharded_chain_decide(models, 4, k, 2, fake, fake, fake, 256, 19008, 0, 8, binding.BF16, f32(1.0), fake, null,
                                           fake, null, fake, null, fake, 1 << 40, null)
    assert st == binding.ERR_INVALID_ARG                # no gather records
    st = lib.polyspec_sharded_chain_pick(models, 4, k, 2, fake, 256, 19008, 0, 8, binding.BF16, f32(-1.0), fake, fake, null, fake, 1 << 40, null)
    assert st == binding.ERR_INVALID_ARG                # temperature
    assert lib.polyspec_sharded_chain_handoff(4, k, 3, 256, fake, fake, fake, fake, null, null, null) == binding.ERR_INVALID_ARG
    assert lib.polyspec_sharded_chain_handoff(4, k, 0, 256, fake, null, fake, fake, null, null, null) == binding.ERR_INVALID_ARG


def test_binding_raises_when_the_library_is_missing(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libpolyspec.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load_library()


def test_package_and_library_versions_agree():
    import paper_2510_26527_b200 as pkg
    major, minor, patch = (int(x) for x in pkg.__version__.split("."))
    assert binding.load_library().polyspec_version() == major * 1000 + minor * 100 + patch * 10
