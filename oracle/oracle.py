"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE, not the product).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
module.  It loads ``libpolyspec_oracle.so`` (built from ``polyspec_oracle.c`` with
gcc), loops over the sequences of a batch and hands each one to the C routines,
which hold all of the arithmetic.  Nothing here touches CUDA or the product
package.

Buffers are CPU tensors (torch float32 / bfloat16 / float64) or numpy arrays
(float32, float64, or uint16 holding bf16 bit patterns), C-contiguous.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "polyspec_oracle.c")
_LIB = os.path.join(_HERE, "libpolyspec_oracle.so")

F32, BF16, F64 = 0, 1, 2
STATUS_NAMES = {0: "ok", 1: "nan_or_posinf_logit", 2: "no_finite_logit", 3: "token_out_of_range", 4: "bad_argument"}

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-std=c99", "-Wall", "-Wextra", "-shared", "-fPIC",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i32p, f32p, f64p = ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_double)
        lib.pso_softmax_row.restype = ctypes.c_int
        lib.pso_softmax_row.argtypes = [vp, ctypes.c_int, ctypes.c_int64, ctypes.c_double, f64p]
        lib.pso_verify_level_seq.restype = ctypes.c_int
        lib.pso_verify_level_seq.argtypes = [vp, vp, ctypes.c_int, ctypes.c_int64, ctypes.c_int,
                                             i32p, f32p, ctypes.c_float, ctypes.c_double,
                                             i32p, i32p, f64p, f64p, f64p, f64p, i32p, f64p]
        lib.pso_verify_chain_seq.restype = ctypes.c_int
        lib.pso_verify_chain_seq.argtypes = [ctypes.POINTER(vp), i32p, ctypes.c_int, i32p, i32p, ctypes.c_int,
                                             f32p, ctypes.c_int64, ctypes.c_int, ctypes.c_int64, ctypes.c_int,
                                             ctypes.c_double, i32p, i32p, i32p, i32p, f64p, f64p, i32p, f64p]
        lib.pso_verify_chain_greedy_seq.restype = ctypes.c_int
        lib.pso_verify_chain_greedy_seq.argtypes = [ctypes.POINTER(vp), i32p, ctypes.c_int, i32p, i32p, ctypes.c_int, ctypes.c_int,
                                                    ctypes.c_int64, ctypes.c_int, i32p, i32p, i32p, i32p]
        _lib = lib
    return _lib


def _buf(x):
    """(address, dtype code, shape, element size, keep-alive object) of a CPU buffer."""
    try:
        import torch
    except ImportError:  # pragma: no cover
        torch = None
    if torch is not None and isinstance(x, torch.Tensor):
        if x.device.type != "cpu":
            raise ValueError("the oracle reads CPU buffers only")
        x = x.contiguous()
        code = {torch.float32: F32, torch.bfloat16: BF16, torch.float64: F64}.get(x.dtype)
        if code is None:
            raise TypeError(f"unsupported logits dtype {x.dtype}")
        return x.data_ptr(), code, tuple(x.shape), x.element_size(), x
    x = np.ascontiguousarray(x)
    code = {np.dtype(np.float32): F32, np.dtype(np.uint16): BF16, np.dtype(np.float64): F64}.get(x.dtype)
    if code is None:
        raise TypeError(f"unsupported logits dtype {x.dtype}")
    return x.ctypes.data, code, x.shape, x.itemsize, x


def _i32(x):
    try:
        import torch
        if isinstance(x, torch.Tensor):
            x = x.cpu().numpy()
    except ImportError:  # pragma: no cover
        pass
    return np.ascontiguousarray(x, dtype=np.int32)


def _f32(x):
    try:
        import torch
        if isinstance(x, torch.Tensor):
            x = x.cpu().numpy()
    except ImportError:  # pragma: no cover
        pass
    return np.ascontiguousarray(x, dtype=np.float32)


def _p(a, ty):
    return a.ctypes.data_as(ctypes.POINTER(ty))


def softmax_row(row, temperature: float) -> np.ndarray:
    """Temperature softmax of one logits row, in float64 (Section 3.1)."""
    addr, code, shape, _, keep = _buf(row)
    V = int(np.prod(shape))
    out = np.empty(V, dtype=np.float64)
    st = _load().pso_softmax_row(addr, code, V, float(temperature), _p(out, ctypes.c_double))
    if st:
        raise ValueError(f"softmax_row: {STATUS_NAMES.get(st, st)}")
    del keep
    return out


def _run(fn, items, threads):
    if threads <= 1 or len(items) <= 1:
        for it in items:
            fn(it)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(fn, items))


def verify_level(logits_p, logits_q, draft_tokens, uniforms, temperature, block_len=None, threads=1, seqs=None):
    """One adjacent pair over a batch: Algorithm 1's inner loop plus the replacement/bonus token.

    logits_p [B, k+1, V], logits_q [B, >=k, V], draft_tokens [B, k], uniforms [B, k+1]
    (entries [b, j<k] are the accept uniforms, [b, k] the sampling uniform).
    Returns a dict of numpy arrays; rows of sequences outside ``seqs`` stay at -1 / NaN.
    """
    lib = _load()
    pa, pc, ps, pe, pk = _buf(logits_p)
    qa, qc, qs, qe, qk = _buf(logits_q)
    if pc != qc:
        raise TypeError("logits_p and logits_q must share a dtype")
    B, rows_p, V = ps
    rows_q = qs[1]
    tok = _i32(draft_tokens)
    k = tok.shape[1]
    u = _f32(uniforms)
    assert u.shape == (B, k + 1) and rows_p >= k + 1 and rows_q >= k and qs[0] == B and qs[2] == V
    bl = np.full(B, k, dtype=np.int32) if block_len is None else _i32(block_len)
    out = {
        "accepted_len": np.full(B, -1, np.int32), "next_token": np.full(B, -1, np.int32),
        "p_at": np.full((B, k), np.nan), "q_at": np.full((B, k), np.nan),
        "accept_margin": np.full((B, k), np.nan), "sample_info": np.zeros((B, 4)),
        "fallback": np.zeros(B, np.int32), "status": np.zeros(B, np.int32),
    }

    def one(b):
        scratch = np.empty(2 * V, dtype=np.float64)
        a = ctypes.c_int32(-1)
        nx = ctypes.c_int32(-1)
        fb = ctypes.c_int32(0)
        st = lib.pso_verify_level_seq(
            pa + b * rows_p * V * pe, qa + b * rows_q * V * qe, pc, V, int(bl[b]),
            _p(tok[b], ctypes.c_int32), _p(u[b], ctypes.c_float), float(u[b, k]), float(temperature),
            ctypes.byref(a), ctypes.byref(nx),
            _p(out["p_at"][b], ctypes.c_double), _p(out["q_at"][b], ctypes.c_double),
            _p(out["accept_margin"][b], ctypes.c_double), _p(out["sample_info"][b], ctypes.c_double),
            ctypes.byref(fb), _p(scratch, ctypes.c_double))
        out["accepted_len"][b], out["next_token"][b] = a.value, nx.value
        out["fallback"][b], out["status"][b] = fb.value, st

    _run(one, list(range(B)) if seqs is None else list(seqs), threads)
    del pk, qk
    return out


def verify_chain(models, k, draft_tokens, uniforms, temperature, bottom_len=None, threads=1, seqs=None):
    """The chain over a batch (Section 3.1: checked bottom-up, by M_{n-1} first and M_1 last).

    models[i] is [B, rows_i, V] (models[0] = M_1, the target; models[-1] = M_n, the drafter),
    k[l] the largest block level l verifies (l = 0 is M_1's level), draft_tokens
    [B, k[-1]], uniforms [n-1, B, kmax+1] with the sampling uniform in slot kmax.
    Returns per-level arrays shaped [n-1, B, ...]; sequences outside ``seqs`` stay at -1.
    """
    lib = _load()
    n = len(models)
    L = n - 1
    bufs = [_buf(m) for m in models]
    code = bufs[0][1]
    assert all(b[1] == code for b in bufs)
    B, _, V = bufs[0][2]
    k = np.ascontiguousarray(k, dtype=np.int32)
    assert k.shape == (L,)
    kmax = int(k.max())
    tok = _i32(draft_tokens)
    u = _f32(uniforms)
    assert u.shape == (L, B, kmax + 1), (u.shape, (L, B, kmax + 1))
    assert tok.shape == (B, int(k[-1]))
    nrows = np.array([b[2][1] for b in bufs], dtype=np.int32)
    bl = np.full(B, int(k[-1]), np.int32) if bottom_len is None else _i32(bottom_len)
    out = {
        "accepted_len": np.full((L, B), -1, np.int32), "block_len": np.full((L, B), -1, np.int32),
        "out_tokens": np.full((L, B, kmax + 1), -1, np.int32), "out_len": np.full((L, B), -1, np.int32),
        "accept_margin": np.full((L, B, kmax), np.nan), "sample_info": np.zeros((L, B, 4)),
        "fallback": np.zeros((L, B), np.int32), "status": np.zeros(B, np.int32),
    }

    def one(b):
        ptrs = (ctypes.c_void_p * n)(*[bufs[i][0] + b * int(nrows[i]) * V * bufs[i][3] for i in range(n)])
        acc = np.empty(L, np.int32); blk = np.empty(L, np.int32); olen = np.empty(L, np.int32)
        otok = np.empty((L, kmax + 1), np.int32)
        marg = np.empty((L, kmax), np.float64); sinfo = np.zeros((L, 4), np.float64)
        fb = np.zeros(L, np.int32)
        ub = np.ascontiguousarray(u[:, b, :])           # [L, kmax+1]
        scratch = np.empty(2 * V, dtype=np.float64)
        st = lib.pso_verify_chain_seq(
            ptrs, _p(nrows, ctypes.c_int32), n, _p(k, ctypes.c_int32), _p(tok[b], ctypes.c_int32), int(bl[b]),
            _p(ub, ctypes.c_float), kmax + 1, kmax, V, code, float(temperature),
            _p(acc, ctypes.c_int32), _p(blk, ctypes.c_int32), _p(otok, ctypes.c_int32), _p(olen, ctypes.c_int32),
            _p(marg, ctypes.c_double), _p(sinfo, ctypes.c_double), _p(fb, ctypes.c_int32),
            _p(scratch, ctypes.c_double))
        out["accepted_len"][:, b] = acc; out["block_len"][:, b] = blk; out["out_len"][:, b] = olen
        out["out_tokens"][:, b, :] = otok; out["accept_margin"][:, b, :] = marg
        out["sample_info"][:, b, :] = sinfo; out["fallback"][:, b] = fb; out["status"][b] = st

    _run(one, list(range(B)) if seqs is None else list(seqs), threads)
    del bufs
    return out


def verify_chain_greedy(models, k, draft_tokens, bottom_len=None, threads=1, seqs=None):
    """The chain under greedy matching (Sections 3.1 and 4.5): a token is accepted iff it is the
    verifier's arg max, the emitted token is the verifier's arg max after the accepted prefix.

    models as in verify_chain; the last one (the drafter's logits) is not read and may be None.
    Returns accepted_len, block_len, out_len [n-1, B], out_tokens [n-1, B, kmax+1], status [B].
    """
    lib = _load()
    n = len(models)
    L = n - 1
    bufs = [_buf(m) if m is not None else None for m in models]
    code = bufs[0][1]
    B, _, V = bufs[0][2]
    k = np.ascontiguousarray(k, dtype=np.int32)
    kmax = int(k.max())
    tok = _i32(draft_tokens)
    assert tok.shape == (B, int(k[-1]))
    nrows = np.array([b[2][1] if b is not None else int(k[-1]) for b in bufs], dtype=np.int32)
    bl = np.full(B, int(k[-1]), np.int32) if bottom_len is None else _i32(bottom_len)
    out = {"accepted_len": np.full((L, B), -1, np.int32), "block_len": np.full((L, B), -1, np.int32),
           "out_tokens": np.full((L, B, kmax + 1), -1, np.int32), "out_len": np.full((L, B), -1, np.int32),
           "status": np.zeros(B, np.int32)}

    def one(b):
        ptrs = (ctypes.c_void_p * n)(*[(bufs[i][0] + b * int(nrows[i]) * V * bufs[i][3]) if bufs[i] is not None else None
                                       for i in range(n)])
        acc = np.empty(L, np.int32); blk = np.empty(L, np.int32); olen = np.empty(L, np.int32)
        otok = np.empty((L, kmax + 1), np.int32)
        st = lib.pso_verify_chain_greedy_seq(ptrs, _p(nrows, ctypes.c_int32), n, _p(k, ctypes.c_int32), _p(tok[b], ctypes.c_int32),
                                             int(bl[b]), kmax, V, code, _p(acc, ctypes.c_int32), _p(blk, ctypes.c_int32),
                                             _p(otok, ctypes.c_int32), _p(olen, ctypes.c_int32))
        out["accepted_len"][:, b] = acc; out["block_len"][:, b] = blk; out["out_len"][:, b] = olen
        out["out_tokens"][:, b, :] = otok; out["status"][b] = st

    _run(one, list(range(B)) if seqs is None else list(seqs), threads)
    del bufs
    return out


def lm_head_logits(hidden, W):
    """logits[b, j, v] = sum_d hidden[b, j, d] * W[v, d] in float64 from the stored bf16 values.

    The last op of a model forward in Algorithm 1 ("p_{1:K} <- M_2(...)", "v <- M_1(...)").
    The contraction itself is the library matmul in float64.
    """
    import torch
    h = hidden.detach().cpu().to(torch.float64)
    w = W.detach().cpu().to(torch.float64)
    return torch.matmul(h, w.t()).contiguous()


def verify_from_hidden(hidden_p, W_p, hidden_q, W_q, draft_tokens, uniforms, temperature,
                       block_len=None, threads=1, seqs=None):
    """Fused-LM-head variant: float64 logits from the bf16 inputs, then verify_level."""
    lp = lm_head_logits(hidden_p, W_p)
    lq = lm_head_logits(hidden_q, W_q)
    out = verify_level(lp, lq, draft_tokens, uniforms, temperature, block_len=block_len, threads=threads, seqs=seqs)
    out["logits_p"], out["logits_q"] = lp, lq
    return out
