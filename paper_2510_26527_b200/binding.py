"""Python front end of libpolyspec's C ABI (include/polyspec.h): argument marshalling only.

Each function here has the name and the arguments of the C entry point it calls; torch
is used for device memory and streams, nothing is computed in Python.  If the CUDA
library cannot be loaded the functions raise: there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpolyspec.so")

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_BAD_INPUT_ON_DEVICE = 1, 2, 3, 4, 5, 6
ERR_SCRATCH_LIMIT = 7
F32, BF16 = 0, 1
MAX_K, MAX_MODELS = 32, 8

EXPORTS = (
    "polyspec_status_string", "polyspec_version", "polyspec_last_cuda_error",
    "polyspec_verify_level_workspace", "polyspec_verify_level",
    "polyspec_verify_chain_workspace", "polyspec_verify_chain",
    "polyspec_chain_row_stats", "polyspec_chain_walk",
    "polyspec_verify_chain_greedy_workspace", "polyspec_verify_chain_greedy",
    "polyspec_verify_chain_host_workspace", "polyspec_verify_chain_host",
    "polyspec_verify_from_hidden_workspace", "polyspec_verify_from_hidden", "polyspec_lm_head",
    "polyspec_from_hidden_project", "polyspec_from_hidden_verify",
    "polyspec_static_scratch_bytes", "polyspec_verify_level_static",
    "polyspec_cost_total_time", "polyspec_cost_insertion", "polyspec_cost_insertion_drafter",
    "polyspec_sharded_level_sizes", "polyspec_sharded_level_stats", "polyspec_sharded_level_decide",
    "polyspec_sharded_level_pick",
    "polyspec_sharded_chain_sizes", "polyspec_sharded_chain_stats", "polyspec_sharded_chain_gather",
    "polyspec_sharded_chain_decide", "polyspec_sharded_chain_pick", "polyspec_sharded_chain_handoff",
    "polyspec_staged_init", "polyspec_staged_round_begin", "polyspec_staged_accumulate", "polyspec_staged_commit",
)


class PolyspecError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = ""
        if status == ERR_CUDA and _lib is not None:
            detail = ": " + _lib.polyspec_last_cuda_error().decode()
        super().__init__(f"{where}: {status_string(status)} (status {status}){detail}")


class ModelLogits(ctypes.Structure):
    _fields_ = [("logits", ctypes.c_void_p), ("rows", ctypes.c_int)]


STAGED_ARRAYS = ("t", "cnt", "rounds", "cycles", "n_committed", "done", "accepted", "committed", "presented", "per_cycle", "remaining")
STAGED_FINISHED, STAGED_EXHAUSTED, STAGED_BAD_INPUT = 1, 2, 3


class StagedState(ctypes.Structure):
    """polyspec_staged_state: sizes, then the device pointers of the state arrays in STAGED_ARRAYS order."""
    _fields_ = [(n, ctypes.c_int) for n in ("B", "K", "mu", "kcap", "N", "R", "C", "cap", "n_tokens")] + \
               [(n, ctypes.c_void_p) for n in STAGED_ARRAYS]


_lib = None


def load_library() -> ctypes.CDLL:
    """Load libpolyspec.so from the package directory; raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2510_26527_b200.buildlib` "
                           "(needs nvcc); libpolyspec has no CPU fallback")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32p, f32p = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
    ci, cf, sz = ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    szp, cip = ctypes.POINTER(ctypes.c_size_t), ctypes.POINTER(ctypes.c_int)
    lib.polyspec_status_string.restype = ctypes.c_char_p
    lib.polyspec_status_string.argtypes = [ci]
    lib.polyspec_last_cuda_error.restype = ctypes.c_char_p
    lib.polyspec_last_cuda_error.argtypes = []
    lib.polyspec_version.restype = ci
    lib.polyspec_version.argtypes = []
    lib.polyspec_verify_level_workspace.restype = ci
    lib.polyspec_verify_level_workspace.argtypes = [ci, ci, ci, ci, szp]
    lib.polyspec_verify_level.restype = ci
    lib.polyspec_verify_level.argtypes = [vp, vp, i32p, f32p, i32p, ci, ci, ci, ci, cf,
                                          i32p, i32p, f32p, f32p, i32p, vp, sz, vp]
    lib.polyspec_verify_chain_workspace.restype = ci
    lib.polyspec_verify_chain_workspace.argtypes = [ci, cip, cip, ci, ci, ci, szp]
    lib.polyspec_verify_chain.restype = ci
    lib.polyspec_verify_chain.argtypes = [ctypes.POINTER(ModelLogits), ci, cip, i32p, f32p, ci, ci, ci, cf,
                                          i32p, i32p, i32p, i32p, i32p, vp, sz, vp]
    lib.polyspec_verify_chain_greedy_workspace.restype = ci
    lib.polyspec_verify_chain_greedy_workspace.argtypes = [ci, cip, cip, ci, ci, ci, szp]
    lib.polyspec_verify_chain_greedy.restype = ci
    lib.polyspec_verify_chain_greedy.argtypes = [ctypes.POINTER(ModelLogits), ci, cip, i32p, ci, ci, ci,
                                                 i32p, i32p, i32p, i32p, i32p, vp, sz, vp]
    lib.polyspec_chain_row_stats.restype = ci
    lib.polyspec_chain_row_stats.argtypes = [ctypes.POINTER(ModelLogits), ci, cip, ci, ci, ci, cf, i32p, vp, sz, vp]
    lib.polyspec_chain_walk.restype = ci
    lib.polyspec_chain_walk.argtypes = lib.polyspec_verify_chain.argtypes
    lib.polyspec_verify_chain_host_workspace.restype = ci
    lib.polyspec_verify_chain_host_workspace.argtypes = [ci, cip, cip, ci, ci, ci, szp]
    lib.polyspec_verify_chain_host.restype = ci
    lib.polyspec_verify_chain_host.argtypes = [ctypes.POINTER(ModelLogits), ci, cip, i32p, f32p, ci, ci, ci, cf,
                                               i32p, i32p, i32p, i32p, i32p, vp, sz, vp]
    lib.polyspec_verify_from_hidden_workspace.restype = ci
    lib.polyspec_verify_from_hidden_workspace.argtypes = [ci, ci, ci, ci, ci, szp]
    lib.polyspec_verify_from_hidden.restype = ci
    lib.polyspec_verify_from_hidden.argtypes = [vp, vp, vp, vp, ci, i32p, f32p, i32p, ci, ci, ci, ci, ci, cf,
                                                i32p, i32p, f32p, f32p, i32p, vp, sz, vp]
    lib.polyspec_from_hidden_project.restype = ci
    lib.polyspec_from_hidden_project.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, i32p, vp, sz, vp]
    lib.polyspec_from_hidden_verify.restype = ci
    lib.polyspec_from_hidden_verify.argtypes = [ci, i32p, f32p, i32p, ci, ci, ci, ci, ci, cf, i32p, i32p, f32p, f32p, i32p, vp, sz, vp]
    lib.polyspec_lm_head.restype = ci
    lib.polyspec_lm_head.argtypes = [vp, vp, ci, ci, ci, f32p, i32p, vp]
    lib.polyspec_cost_total_time.restype = ctypes.c_double
    lib.polyspec_cost_total_time.argtypes = [ci, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double), ctypes.c_double, ctypes.c_double]
    lib.polyspec_cost_insertion.restype = ci
    lib.polyspec_cost_insertion.argtypes = [ctypes.c_double] * 5 + [ctypes.POINTER(ctypes.c_double)] * 2
    lib.polyspec_cost_insertion_drafter.restype = ci
    lib.polyspec_cost_insertion_drafter.argtypes = [ctypes.c_double] * 5 + [ctypes.POINTER(ctypes.c_double)] * 2
    lib.polyspec_static_scratch_bytes.restype = sz
    lib.polyspec_static_scratch_bytes.argtypes = []
    lib.polyspec_verify_level_static.restype = ci
    lib.polyspec_verify_level_static.argtypes = [vp, vp, i32p, f32p, i32p, ci, ci, ci, ci, cf,
                                                 i32p, i32p, f32p, f32p, i32p, vp]
    lib.polyspec_sharded_level_sizes.restype = ci
    lib.polyspec_sharded_level_sizes.argtypes = [ci, ci, ci, ci, ci, szp, szp, szp]
    lib.polyspec_sharded_level_stats.restype = ci
    lib.polyspec_sharded_level_stats.argtypes = [vp, vp, i32p, ci, ci, ci, ci, ci, ci, cf, vp, i32p, vp, sz, vp]
    lib.polyspec_sharded_level_decide.restype = ci
    lib.polyspec_sharded_level_decide.argtypes = [vp, vp, i32p, f32p, i32p, ci, ci, ci, ci, ci, ci, cf, vp,
                                                  i32p, f32p, f32p, vp, i32p, vp, sz, vp]
    lib.polyspec_sharded_level_pick.restype = ci
    lib.polyspec_sharded_level_pick.argtypes = [vp, vp, f32p, ci, ci, ci, ci, ci, ci, cf, vp, i32p, i32p, vp, sz, vp]
    mlp = ctypes.POINTER(ModelLogits)
    lib.polyspec_sharded_chain_sizes.restype = ci
    lib.polyspec_sharded_chain_sizes.argtypes = [ci, cip, cip, ci, ci, ci, ci, szp, szp, szp, szp]
    lib.polyspec_sharded_chain_stats.restype = ci
    lib.polyspec_sharded_chain_stats.argtypes = [mlp, ci, cip, ci, ci, ci, ci, ci, cf, vp, i32p, vp, sz, vp]
    lib.polyspec_sharded_chain_gather.restype = ci
    lib.polyspec_sharded_chain_gather.argtypes = [mlp, ci, cip, ci, i32p, i32p, ci, ci, ci, ci, ci, vp, vp, sz, vp]
    lib.polyspec_sharded_chain_decide.restype = ci
    lib.polyspec_sharded_chain_decide.argtypes = [mlp, ci, cip, ci, i32p, i32p, f32p, ci, ci, ci, ci, ci, cf, vp, vp, i32p, i32p, vp,
                                                  i32p, vp, sz, vp]
    lib.polyspec_sharded_chain_pick.restype = ci
    lib.polyspec_sharded_chain_pick.argtypes = [mlp, ci, cip, ci, f32p, ci, ci, ci, ci, ci, cf, vp, i32p, i32p, vp, sz, vp]
    lib.polyspec_sharded_chain_handoff.restype = ci
    lib.polyspec_sharded_chain_handoff.argtypes = [ci, cip, ci, ci, i32p, i32p, i32p, i32p, i32p, i32p, vp]
    ssp = ctypes.POINTER(StagedState)
    lib.polyspec_staged_init.restype = ci
    lib.polyspec_staged_init.argtypes = [ssp, vp]
    lib.polyspec_staged_round_begin.restype = ci
    lib.polyspec_staged_round_begin.argtypes = [ssp, i32p, f32p, i32p, i32p, f32p, i32p, vp]
    lib.polyspec_staged_accumulate.restype = ci
    lib.polyspec_staged_accumulate.argtypes = [ssp, i32p, i32p, i32p, i32p, f32p, i32p, i32p, f32p, i32p, vp]
    lib.polyspec_staged_commit.restype = ci
    lib.polyspec_staged_commit.argtypes = [ssp, i32p, i32p, i32p, vp]
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().polyspec_status_string(int(status)).decode()


def version() -> int:
    return load_library().polyspec_version()


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"logits must be float32 or bfloat16, got {t.dtype}")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(st: int, where: str):
    if st != OK:
        raise PolyspecError(st, where)


def _dev_check(*tensors):
    for t in tensors:
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise ValueError("device-pointer arguments must be contiguous CUDA tensors")


def _workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


# ------------------------------------------------------------------ verify_level
def polyspec_verify_level_workspace(B: int, k: int, V: int, dt: int) -> int:
    n = ctypes.c_size_t(0)
    _check(load_library().polyspec_verify_level_workspace(B, k, V, dt, ctypes.byref(n)), "polyspec_verify_level_workspace")
    return n.value


def polyspec_verify_level(logits_p, logits_q, draft_tokens, uniforms, temperature, block_len=None,
                          want_probs=False, workspace=None, out=None, device_status=None, stream=None):
    """One adjacent pair over a batch.  logits_p [B,k+1,V], logits_q [B,k,V], draft_tokens [B,k] int32,
    uniforms [B,k+1] float32; returns device tensors accepted_len [B], next_token [B] (and p_at_draft,
    q_at_draft [B,k] if want_probs) plus the device status word."""
    lib = load_library()
    _dev_check(logits_p, logits_q, draft_tokens, uniforms, block_len)
    B, rows_p, V = logits_p.shape
    k = draft_tokens.shape[1]
    if rows_p != k + 1 or tuple(logits_q.shape) != (B, k, V) or tuple(uniforms.shape) != (B, k + 1):
        raise ValueError("shapes must be logits_p [B,k+1,V], logits_q [B,k,V], draft_tokens [B,k], uniforms [B,k+1]")
    if draft_tokens.dtype != torch.int32 or uniforms.dtype != torch.float32 or logits_q.dtype != logits_p.dtype:
        raise TypeError("draft_tokens int32, uniforms float32, logits_p/logits_q one dtype")
    dev = logits_p.device
    dt = _dt(logits_p)
    if workspace is None:
        workspace = _workspace(polyspec_verify_level_workspace(B, k, V, dt), dev)
    if out is None:
        out = {"accepted_len": torch.empty(B, dtype=torch.int32, device=dev),
               "next_token": torch.empty(B, dtype=torch.int32, device=dev)}
        if want_probs:
            out["p_at_draft"] = torch.empty((B, k), dtype=torch.float32, device=dev)
            out["q_at_draft"] = torch.empty((B, k), dtype=torch.float32, device=dev)
    if device_status is None:
        device_status = torch.zeros(1, dtype=torch.int32, device=dev)
    st = lib.polyspec_verify_level(
        _ptr(logits_p), _ptr(logits_q), _ptr(draft_tokens), _ptr(uniforms), _ptr(block_len),
        B, k, V, dt, float(temperature), _ptr(out["accepted_len"]), _ptr(out["next_token"]),
        _ptr(out.get("p_at_draft")), _ptr(out.get("q_at_draft")), _ptr(device_status),
        _ptr(workspace), workspace.numel(), _stream(stream))
    _check(st, "polyspec_verify_level")
    out["device_status"] = device_status
    return out


# ------------------------------------------------------------------ verify_chain
def _int_array(vals: Sequence[int]):
    return (ctypes.c_int * len(vals))(*[int(v) for v in vals])


def polyspec_verify_chain_workspace(k: Sequence[int], rows: Sequence[int], B: int, V: int, dt: int) -> int:
    n = ctypes.c_size_t(0)
    _check(load_library().polyspec_verify_chain_workspace(len(rows), _int_array(k), _int_array(rows), B, V, dt, ctypes.byref(n)),
           "polyspec_verify_chain_workspace")
    return n.value


def chain_outputs(L: int, B: int, kmax: int, device, pin=False) -> dict:
    kw = {"dtype": torch.int32, "device": device}
    if pin:
        kw["pin_memory"] = True
    return {"accepted_len": torch.empty((L, B), **kw), "block_len": torch.empty((L, B), **kw),
            "out_tokens": torch.empty((L, B, kmax + 1), **kw), "out_len": torch.empty((L, B), **kw)}


def polyspec_verify_chain(models, k, draft_tokens, uniforms, temperature, workspace=None, out=None,
                          device_status=None, stream=None):
    """n models (models[0] = M_1 ... models[-1] = M_n, each [B, rows_i, V]), n-1 levels verified bottom-up.
    k[l] = largest block level l verifies; draft_tokens [B, k[-1]]; uniforms [n-1, B, max(k)+1]."""
    lib = load_library()
    _dev_check(*models, draft_tokens, uniforms)
    n = len(models)
    L = n - 1
    B, _, V = models[0].shape
    dt = _dt(models[0])
    rows = [int(m.shape[1]) for m in models]
    kmax = max(int(x) for x in k)
    if any(m.dtype != models[0].dtype or m.shape[0] != B or m.shape[2] != V for m in models):
        raise ValueError("all models must share dtype, batch and vocabulary")
    if tuple(uniforms.shape) != (L, B, kmax + 1) or tuple(draft_tokens.shape) != (B, int(k[-1])):
        raise ValueError("uniforms must be [n-1, B, max(k)+1] and draft_tokens [B, k[-1]]")
    if draft_tokens.dtype != torch.int32 or uniforms.dtype != torch.float32:
        raise TypeError("draft_tokens int32, uniforms float32")
    dev = models[0].device
    if workspace is None:
        workspace = _workspace(polyspec_verify_chain_workspace(k, rows, B, V, dt), dev)
    if out is None:
        out = chain_outputs(L, B, kmax, dev)
    if device_status is None:
        device_status = torch.zeros(1, dtype=torch.int32, device=dev)
    arr = (ModelLogits * n)(*[ModelLogits(m.data_ptr(), r) for m, r in zip(models, rows)])
    st = lib.polyspec_verify_chain(arr, n, _int_array(k), _ptr(draft_tokens), _ptr(uniforms), B, V, dt, float(temperature),
                                   _ptr(out["accepted_len"]), _ptr(out["block_len"]), _ptr(out["out_tokens"]),
                                   _ptr(out["out_len"]), _ptr(device_status), _ptr(workspace), workspace.numel(),
                                   _stream(stream))
    _check(st, "polyspec_verify_chain")
    out["device_status"] = device_status
    return out


def polyspec_verify_chain_greedy_workspace(k: Sequence[int], rows: Sequence[int], B: int, V: int, dt: int) -> int:
    n = ctypes.c_size_t(0)
    _check(load_library().polyspec_verify_chain_greedy_workspace(len(rows), _int_array(k), _int_array(rows), B, V, dt, ctypes.byref(n)),
           "polyspec_verify_chain_greedy_workspace")
    return n.value


def polyspec_verify_chain_greedy(models, k, draft_tokens, workspace=None, out=None, device_status=None, stream=None):
    """The chain under greedy matching.  models as in polyspec_verify_chain; the last entry (the drafter's logits)
    is not read and may be None.  Returns the same four outputs plus the device status word."""
    lib = load_library()
    verifiers = list(models[:-1])
    _dev_check(*verifiers, draft_tokens)
    n = len(models)
    L = n - 1
    B, _, V = verifiers[0].shape
    dt = _dt(verifiers[0])
    rows = [int(m.shape[1]) for m in verifiers] + [int(k[-1])]
    kmax = max(int(x) for x in k)
    if any(m.dtype != verifiers[0].dtype or m.shape[0] != B or m.shape[2] != V for m in verifiers):
        raise ValueError("all verifiers must share dtype, batch and vocabulary")
    if tuple(draft_tokens.shape) != (B, int(k[-1])) or draft_tokens.dtype != torch.int32:
        raise ValueError("draft_tokens must be int32 [B, k[-1]]")
    dev = verifiers[0].device
    if workspace is None:
        workspace = _workspace(polyspec_verify_chain_greedy_workspace(k, rows, B, V, dt), dev)
    if out is None:
        out = chain_outputs(L, B, kmax, dev)
    if device_status is None:
        device_status = torch.zeros(1, dtype=torch.int32, device=dev)
    ptrs = [m.data_ptr() for m in verifiers] + [models[-1].data_ptr() if models[-1] is not None else None]
    arr = (ModelLogits * n)(*[ModelLogits(pt, r) for pt, r in zip(ptrs, rows)])
    with torch.cuda.device(dev):
        st = lib.polyspec_verify_chain_greedy(arr, n, _int_array(k), _ptr(draft_tokens), B, V, dt,
                                              _ptr(out["accepted_len"]), _ptr(out["block_len"]), _ptr(out["out_tokens"]),
                                              _ptr(out["out_len"]), _ptr(device_status), _ptr(workspace), workspace.numel(),
                                              _stream(stream))
    _check(st, "polyspec_verify_chain_greedy")
    out["device_status"] = device_status
    return out


class ChainCall:
    """A prepared polyspec_verify_chain call: arguments marshalled once, outputs and workspace allocated once.

    launch() is the single C-ABI call; row_stats() and walk() are its two halves
    (polyspec_chain_row_stats / polyspec_chain_walk)."""

    def __init__(self, models, k, draft_tokens, uniforms, temperature, stream=None):
        self.lib = load_library()
        _dev_check(*models, draft_tokens, uniforms)
        self.models, self.draft_tokens, self.uniforms = list(models), draft_tokens, uniforms
        self.n = len(models)
        self.B, _, self.V = models[0].shape
        self.dt = _dt(models[0])
        self.rows = [int(m.shape[1]) for m in models]
        self.k = [int(x) for x in k]
        self.kmax = max(self.k)
        self.temperature = float(temperature)
        dev = models[0].device
        self.workspace = _workspace(polyspec_verify_chain_workspace(self.k, self.rows, self.B, self.V, self.dt), dev)
        self.out = chain_outputs(self.n - 1, self.B, self.kmax, dev)
        self.device_status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.out["device_status"] = self.device_status
        self._arr = (ModelLogits * self.n)(*[ModelLogits(m.data_ptr(), r) for m, r in zip(models, self.rows)])
        self._k = _int_array(self.k)
        self.stream = stream

    def _tail(self):
        o = self.out
        return (_ptr(o["accepted_len"]), _ptr(o["block_len"]), _ptr(o["out_tokens"]), _ptr(o["out_len"]),
                _ptr(self.device_status), _ptr(self.workspace), self.workspace.numel(), _stream(self.stream))

    def launch(self):
        _check(self.lib.polyspec_verify_chain(self._arr, self.n, self._k, _ptr(self.draft_tokens), _ptr(self.uniforms),
                                              self.B, self.V, self.dt, self.temperature, *self._tail()), "polyspec_verify_chain")
        return self.out

    def row_stats(self):
        _check(self.lib.polyspec_chain_row_stats(self._arr, self.n, self._k, self.B, self.V, self.dt, self.temperature,
                                                 _ptr(self.device_status), _ptr(self.workspace), self.workspace.numel(), _stream(self.stream)),
               "polyspec_chain_row_stats")

    def walk(self):
        _check(self.lib.polyspec_chain_walk(self._arr, self.n, self._k, _ptr(self.draft_tokens), _ptr(self.uniforms),
                                            self.B, self.V, self.dt, self.temperature, *self._tail()), "polyspec_chain_walk")
        return self.out


def polyspec_verify_chain_host_workspace(k: Sequence[int], rows: Sequence[int], B: int, V: int, dt: int) -> int:
    n = ctypes.c_size_t(0)
    _check(load_library().polyspec_verify_chain_host_workspace(len(rows), _int_array(k), _int_array(rows), B, V, dt, ctypes.byref(n)),
           "polyspec_verify_chain_host_workspace")
    return n.value


def polyspec_verify_chain_host(models, k, draft_tokens, uniforms, temperature, workspace, out=None,
                               host_status=None, stream=None):
    """The chain for HOST buffers (CPU tensors, ideally pinned); `workspace` is a device tensor of at least
    polyspec_verify_chain_host_workspace bytes.  Outputs are CPU tensors, valid after the stream synchronises."""
    lib = load_library()
    n = len(models)
    L = n - 1
    B, _, V = models[0].shape
    dt = _dt(models[0])
    rows = [int(m.shape[1]) for m in models]
    kmax = max(int(x) for x in k)
    for t in list(models) + [draft_tokens, uniforms]:
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("polyspec_verify_chain_host takes contiguous CPU tensors")
    if not workspace.is_cuda:
        raise ValueError("the workspace must be a CUDA tensor")
    if out is None:
        out = chain_outputs(L, B, kmax, "cpu", pin=True)
    if host_status is None:
        host_status = torch.zeros(1, dtype=torch.int32, pin_memory=True)
    arr = (ModelLogits * n)(*[ModelLogits(m.data_ptr(), r) for m, r in zip(models, rows)])
    with torch.cuda.device(workspace.device):
        st = lib.polyspec_verify_chain_host(arr, n, _int_array(k), _ptr(draft_tokens), _ptr(uniforms), B, V, dt,
                                            float(temperature), _ptr(out["accepted_len"]), _ptr(out["block_len"]),
                                            _ptr(out["out_tokens"]), _ptr(out["out_len"]), _ptr(host_status),
                                            _ptr(workspace), workspace.numel(), _stream(stream))
    _check(st, "polyspec_verify_chain_host")
    out["host_status"] = host_status
    return out


# ------------------------------------------------------------------ verify_from_hidden
def polyspec_verify_from_hidden_workspace(B: int, k: int, V: int, d_p: int, d_q: int) -> int:
    n = ctypes.c_size_t(0)
    _check(load_library().polyspec_verify_from_hidden_workspace(B, k, V, d_p, d_q, ctypes.byref(n)),
           "polyspec_verify_from_hidden_workspace")
    return n.value


def polyspec_verify_from_hidden(hidden_p, W_p, hidden_q, W_q, draft_tokens, uniforms, temperature, block_len=None,
                                want_probs=False, workspace=None, out=None, device_status=None, stream=None):
    """verify_level with the LM-head projection fused in front: hidden_p [B,k+1,d_p], W_p [V,d_p],
    hidden_q [B,rows_q>=k,d_q], W_q [V,d_q], all bf16."""
    lib = load_library()
    _dev_check(hidden_p, W_p, hidden_q, W_q, draft_tokens, uniforms, block_len)
    B, rows_p, d_p = hidden_p.shape
    _, rows_q, d_q = hidden_q.shape
    V = W_p.shape[0]
    k = draft_tokens.shape[1]
    if rows_p != k + 1 or W_q.shape[0] != V or W_p.shape[1] != d_p or W_q.shape[1] != d_q or hidden_q.shape[0] != B:
        raise ValueError("shapes must be hidden_p [B,k+1,d_p], W_p [V,d_p], hidden_q [B,rows_q,d_q], W_q [V,d_q]")
    if any(t.dtype != torch.bfloat16 for t in (hidden_p, W_p, hidden_q, W_q)):
        raise TypeError("hidden states and LM-head weights must be bfloat16")
    dev = hidden_p.device
    if workspace is None:
        workspace = _workspace(polyspec_verify_from_hidden_workspace(B, k, V, d_p, d_q), dev)
    if out is None:
        out = {"accepted_len": torch.empty(B, dtype=torch.int32, device=dev),
               "next_token": torch.empty(B, dtype=torch.int32, device=dev)}
        if want_probs:
            out["p_at_draft"] = torch.empty((B, k), dtype=torch.float32, device=dev)
            out["q_at_draft"] = torch.empty((B, k), dtype=torch.float32, device=dev)
    if device_status is None:
        device_status = torch.zeros(1, dtype=torch.int32, device=dev)
    st = lib.polyspec_verify_from_hidden(
        _ptr(hidden_p), _ptr(W_p), _ptr(hidden_q), _ptr(W_q), rows_q, _ptr(draft_tokens), _ptr(uniforms), _ptr(block_len),
        B, k, V, d_p, d_q, float(temperature), _ptr(out["accepted_len"]), _ptr(out["next_token"]),
        _ptr(out.get("p_at_draft")), _ptr(out.get("q_at_draft")), _ptr(device_status),
        _ptr(workspace), workspace.numel(), _stream(stream))
    _check(st, "polyspec_verify_from_hidden")
    out["device_status"] = device_status
    return out


class FusedCall:
    """A prepared polyspec_verify_from_hidden call: arguments marshalled once, outputs and workspace allocated once.

    launch() is the single C-ABI call; project() and verify() are its two halves
    (polyspec_from_hidden_project / polyspec_from_hidden_verify)."""

    def __init__(self, hidden_p, W_p, hidden_q, W_q, draft_tokens, uniforms, temperature, block_len=None, stream=None):
        self.lib = load_library()
        _dev_check(hidden_p, W_p, hidden_q, W_q, draft_tokens, uniforms, block_len)
        if any(t.dtype != torch.bfloat16 for t in (hidden_p, W_p, hidden_q, W_q)):
            raise TypeError("hidden states and LM-head weights must be bfloat16")
        self.t = (hidden_p, W_p, hidden_q, W_q, draft_tokens, uniforms, block_len)
        self.B, rows_p, self.d_p = hidden_p.shape
        _, self.rows_q, self.d_q = hidden_q.shape
        self.V = W_p.shape[0]
        self.k = draft_tokens.shape[1]
        if rows_p != self.k + 1 or W_q.shape[0] != self.V or W_p.shape[1] != self.d_p or W_q.shape[1] != self.d_q:
            raise ValueError("shapes must be hidden_p [B,k+1,d_p], W_p [V,d_p], hidden_q [B,rows_q,d_q], W_q [V,d_q]")
        self.temperature = float(temperature)
        dev = hidden_p.device
        self.workspace = _workspace(polyspec_verify_from_hidden_workspace(self.B, self.k, self.V, self.d_p, self.d_q), dev)
        self.out = {"accepted_len": torch.empty(self.B, dtype=torch.int32, device=dev),
                    "next_token": torch.empty(self.B, dtype=torch.int32, device=dev)}
        self.device_status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.out["device_status"] = self.device_status
        self.stream = stream

    def _sizes(self):
        return (self.B, self.k, self.V, self.d_p, self.d_q)

    def launch(self):
        hp, wp, hq, wq, tok, u, bl = self.t
        _check(self.lib.polyspec_verify_from_hidden(
            _ptr(hp), _ptr(wp), _ptr(hq), _ptr(wq), self.rows_q, _ptr(tok), _ptr(u), _ptr(bl), *self._sizes(), self.temperature,
            _ptr(self.out["accepted_len"]), _ptr(self.out["next_token"]), None, None, _ptr(self.device_status),
            _ptr(self.workspace), self.workspace.numel(), _stream(self.stream)), "polyspec_verify_from_hidden")
        return self.out

    def project(self):
        hp, wp, hq, wq, _, _, _ = self.t
        _check(self.lib.polyspec_from_hidden_project(
            _ptr(hp), _ptr(wp), _ptr(hq), _ptr(wq), self.rows_q, *self._sizes(), self.temperature, _ptr(self.device_status),
            _ptr(self.workspace), self.workspace.numel(), _stream(self.stream)), "polyspec_from_hidden_project")

    def verify(self):
        _, _, _, _, tok, u, bl = self.t
        _check(self.lib.polyspec_from_hidden_verify(
            self.rows_q, _ptr(tok), _ptr(u), _ptr(bl), *self._sizes(), self.temperature,
            _ptr(self.out["accepted_len"]), _ptr(self.out["next_token"]), None, None, _ptr(self.device_status),
            _ptr(self.workspace), self.workspace.numel(), _stream(self.stream)), "polyspec_from_hidden_verify")
        return self.out


def polyspec_lm_head(hidden, W, out=None, device_status=None, stream=None):
    """The projection alone: hidden [..., d] bf16, W [V, d] bf16 -> fp32 logits [..., V]."""
    lib = load_library()
    _dev_check(hidden, W, out)
    if hidden.dtype != torch.bfloat16 or W.dtype != torch.bfloat16:
        raise TypeError("hidden states and LM-head weights must be bfloat16")
    d = hidden.shape[-1]
    rows = hidden.numel() // d
    V = W.shape[0]
    if W.shape[1] != d:
        raise ValueError("hidden [..., d] and W [V, d] must share d")
    if out is None:
        out = torch.empty(tuple(hidden.shape[:-1]) + (V,), dtype=torch.float32, device=hidden.device)
    if device_status is None:
        device_status = torch.zeros(1, dtype=torch.int32, device=hidden.device)
    with torch.cuda.device(hidden.device):
        st = lib.polyspec_lm_head(_ptr(hidden), _ptr(W), rows, V, d, _ptr(out), _ptr(device_status), _stream(stream))
    _check(st, "polyspec_lm_head")
    return out, device_status


# ------------------------------------------------------------------ verify_level without a workspace
def polyspec_static_scratch_bytes() -> int:
    return int(load_library().polyspec_static_scratch_bytes())


def polyspec_verify_level_static(logits_p, logits_q, draft_tokens, uniforms, temperature, out, block_len=None,
                                 device_status=None, stream=None):
    """polyspec_verify_level for callers that cannot allocate device memory: no workspace is passed, the
    library's built-in scratch array is used, and this wrapper allocates nothing either -- `out` must hold
    the caller's own accepted_len / next_token (and optionally p_at_draft / q_at_draft) device tensors.
    Raises PolyspecError(ERR_SCRATCH_LIMIT) when the problem needs more than polyspec_static_scratch_bytes()."""
    lib = load_library()
    _dev_check(logits_p, logits_q, draft_tokens, uniforms, block_len)
    B, rows_p, V = logits_p.shape
    k = draft_tokens.shape[1]
    if rows_p != k + 1 or tuple(logits_q.shape) != (B, k, V) or tuple(uniforms.shape) != (B, k + 1):
        raise ValueError("shapes must be logits_p [B,k+1,V], logits_q [B,k,V], draft_tokens [B,k], uniforms [B,k+1]")
    with torch.cuda.device(logits_p.device):
        st = lib.polyspec_verify_level_static(
            _ptr(logits_p), _ptr(logits_q), _ptr(draft_tokens), _ptr(uniforms), _ptr(block_len),
            B, k, V, _dt(logits_p), float(temperature), _ptr(out["accepted_len"]), _ptr(out["next_token"]),
            _ptr(out.get("p_at_draft")), _ptr(out.get("q_at_draft")), _ptr(device_status), _stream(stream))
    _check(st, "polyspec_verify_level_static")
    return out


# ------------------------------------------------------------------ cost model (host arithmetic)
def polyspec_cost_total_time(T: Sequence[float], L: Sequence[float], beta: float, N: float) -> float:
    """Lemma 3.1 (Eq. 3): T = sum_{i<n} (N / L_i) T_i + beta (N / L_{n-1}) T_n."""
    n = len(T)
    if len(L) != n - 1:
        raise ValueError("L must hold n - 1 acceptance lengths")
    Ta = (ctypes.c_double * n)(*[float(x) for x in T])
    La = (ctypes.c_double * max(n - 1, 1))(*[float(x) for x in L])
    return float(load_library().polyspec_cost_total_time(n, Ta, La, float(beta), float(N)))


def polyspec_cost_insertion(T_new: float, T_i: float, L_new: float, L_i: float, L_i_new: float):
    """Theorem 3.2, first condition: (improves, T_new / T_i, L_new (1 / L_i - 1 / L_{i-new}))."""
    lhs, rhs = ctypes.c_double(0.0), ctypes.c_double(0.0)
    r = load_library().polyspec_cost_insertion(float(T_new), float(T_i), float(L_new), float(L_i), float(L_i_new),
                                               ctypes.byref(lhs), ctypes.byref(rhs))
    if r < 0:
        raise ValueError("all five quantities must be positive")
    return bool(r), lhs.value, rhs.value


def polyspec_cost_insertion_drafter(T_new: float, T_next: float, L_new: float, L_i: float, beta: float):
    """Theorem 3.2, second condition (as its proof derives it): (improves, T_new / T_{i+1}, beta (L_new / L_i - 1))."""
    lhs, rhs = ctypes.c_double(0.0), ctypes.c_double(0.0)
    r = load_library().polyspec_cost_insertion_drafter(float(T_new), float(T_next), float(L_new), float(L_i), float(beta),
                                                       ctypes.byref(lhs), ctypes.byref(rhs))
    if r < 0:
        raise ValueError("all five quantities must be positive")
    return bool(r), lhs.value, rhs.value


# ------------------------------------------------------------------ one level, vocabulary sharded over ranks
def polyspec_sharded_level_sizes(B: int, k: int, V_local: int, dt: int, n_ranks: int):
    """(workspace bytes, stats record bytes, mass record bytes) of the sharded level calls."""
    w, a, m = ctypes.c_size_t(0), ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(load_library().polyspec_sharded_level_sizes(B, k, V_local, dt, n_ranks, ctypes.byref(w), ctypes.byref(a), ctypes.byref(m)),
           "polyspec_sharded_level_sizes")
    return w.value, a.value, m.value


class ShardedLevelCall:
    """One rank's side of a vocabulary-sharded level: its slices of the logits, its workspace and records.

    stats() -> this rank's stats record; decide(all ranks' stats records) -> (accepted_len, this rank's mass
    record); pick(all ranks' mass records) -> next_token, -1 unless this rank's slice holds the token.  The
    exchanges between the calls are the caller's (see paper_2510_26527_b200.sharded)."""

    def __init__(self, logits_p, logits_q, draft_tokens, uniforms, temperature, rank, n_ranks, block_len=None,
                 want_probs=False, stream=None):
        self.lib = load_library()
        _dev_check(logits_p, logits_q, draft_tokens, uniforms, block_len)
        self.B, rows_p, self.V_local = logits_p.shape
        self.k = int(draft_tokens.shape[1])
        if rows_p != self.k + 1 or tuple(logits_q.shape) != (self.B, self.k, self.V_local) or logits_q.dtype != logits_p.dtype:
            raise ValueError("shapes must be logits_p [B,k+1,V_local], logits_q [B,k,V_local] of one dtype")
        self.dt = _dt(logits_p)
        self.t = (logits_p, logits_q, draft_tokens, uniforms, block_len)
        self.rank, self.n_ranks = int(rank), int(n_ranks)
        self.temperature = float(temperature)
        dev = logits_p.device
        wbytes, self.stats_bytes, self.mass_bytes = polyspec_sharded_level_sizes(self.B, self.k, self.V_local, self.dt, self.n_ranks)
        self.workspace = _workspace(wbytes, dev)
        self.stats_record = torch.zeros(self.stats_bytes, dtype=torch.uint8, device=dev)
        self.mass_record = torch.zeros(self.mass_bytes, dtype=torch.uint8, device=dev)
        self.accepted_len = torch.empty(self.B, dtype=torch.int32, device=dev)
        self.next_token = torch.empty(self.B, dtype=torch.int32, device=dev)
        self.p_at = torch.zeros((self.B, self.k), dtype=torch.float32, device=dev) if want_probs else None
        self.q_at = torch.zeros((self.B, self.k), dtype=torch.float32, device=dev) if want_probs else None
        self.device_status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.stream = stream

    def _sizes(self):
        return (self.B, self.k, self.V_local, self.rank, self.n_ranks, self.dt, self.temperature)

    def _tail(self):
        return (_ptr(self.device_status), _ptr(self.workspace), self.workspace.numel(), _stream(self.stream))

    def stats(self):
        lp, lq, tok, _, _ = self.t
        _check(self.lib.polyspec_sharded_level_stats(_ptr(lp), _ptr(lq), _ptr(tok), *self._sizes(), _ptr(self.stats_record), *self._tail()),
               "polyspec_sharded_level_stats")
        return self.stats_record

    def decide(self, stats_records):
        lp, lq, tok, u, bl = self.t
        _dev_check(stats_records)
        if stats_records.numel() != self.n_ranks * self.stats_bytes:
            raise ValueError("need every rank's stats record, in rank order")
        _check(self.lib.polyspec_sharded_level_decide(_ptr(lp), _ptr(lq), _ptr(tok), _ptr(u), _ptr(bl), *self._sizes(), _ptr(stats_records),
                                                      _ptr(self.accepted_len), _ptr(self.p_at), _ptr(self.q_at), _ptr(self.mass_record),
                                                      *self._tail()), "polyspec_sharded_level_decide")
        return self.accepted_len, self.mass_record

    def pick(self, mass_records):
        lp, lq, _, u, _ = self.t
        _dev_check(mass_records)
        if mass_records.numel() != self.n_ranks * self.mass_bytes:
            raise ValueError("need every rank's mass record, in rank order")
        _check(self.lib.polyspec_sharded_level_pick(_ptr(lp), _ptr(lq), _ptr(u), *self._sizes(), _ptr(mass_records), _ptr(self.next_token),
                                                    *self._tail()), "polyspec_sharded_level_pick")
        return self.next_token


def polyspec_sharded_chain_sizes(k: Sequence[int], rows: Sequence[int], B: int, V_local: int, dt: int, n_ranks: int):
    """(workspace, stats record, gather record, mass record) bytes of the sharded chain calls."""
    w, a, g, m = (ctypes.c_size_t(0) for _ in range(4))
    _check(load_library().polyspec_sharded_chain_sizes(len(rows), _int_array(k), _int_array(rows), B, V_local, dt, n_ranks,
                                                       ctypes.byref(w), ctypes.byref(a), ctypes.byref(g), ctypes.byref(m)),
           "polyspec_sharded_chain_sizes")
    return w.value, a.value, g.value, m.value


class ShardedChainCall:
    """One rank's side of a vocabulary-sharded chain: its slices of every model's logits, its workspace, records,
    the block being verified and the chain's outputs (identical on every rank once a level is handed off).

    stats() once; then per level, bottom-up: gather(level), decide(level, stats records, gather records),
    pick(level, mass records), handoff(level, token after the max over ranks)."""

    def __init__(self, models, k, draft_tokens, uniforms, temperature, rank, n_ranks, stream=None):
        self.lib = load_library()
        _dev_check(*models, draft_tokens, uniforms)
        self.models = list(models)
        self.n = len(models)
        self.L = self.n - 1
        self.B, _, self.V_local = models[0].shape
        self.dt = _dt(models[0])
        self.rows = [int(m.shape[1]) for m in models]
        self.k = [int(x) for x in k]
        self.kmax = max(self.k)
        if any(m.dtype != models[0].dtype or m.shape[0] != self.B or m.shape[2] != self.V_local for m in models):
            raise ValueError("every model's slice must be [B, rows, V_local] of one dtype")
        if tuple(draft_tokens.shape) != (self.B, self.k[-1]) or tuple(uniforms.shape) != (self.L, self.B, self.kmax + 1):
            raise ValueError("shapes must be draft_tokens [B, k[-1]], uniforms [n_models-1, B, kmax+1]")
        self.rank, self.n_ranks = int(rank), int(n_ranks)
        self.temperature = float(temperature)
        self.uniforms = uniforms
        dev = models[0].device
        wbytes, self.stats_bytes, self.gather_bytes, self.mass_bytes = polyspec_sharded_chain_sizes(
            self.k, self.rows, self.B, self.V_local, self.dt, self.n_ranks)
        self.workspace = _workspace(wbytes, dev)
        self.stats_record = torch.zeros(self.stats_bytes, dtype=torch.uint8, device=dev)
        self.gather_record = torch.zeros(self.gather_bytes, dtype=torch.uint8, device=dev)
        self.mass_record = torch.zeros(self.mass_bytes, dtype=torch.uint8, device=dev)
        self.block_tokens = torch.full((self.B, self.kmax + 1), -1, dtype=torch.int32, device=dev)
        self.block_tokens[:, : self.k[-1]] = draft_tokens
        self.block_len = torch.full((self.B,), self.k[-1], dtype=torch.int32, device=dev)
        self.next_token = torch.empty(self.B, dtype=torch.int32, device=dev)
        self.out = chain_outputs(self.L, self.B, self.kmax, dev)
        self.device_status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.out["device_status"] = self.device_status
        self._arr = (ModelLogits * self.n)(*[ModelLogits(m.data_ptr(), r) for m, r in zip(models, self.rows)])
        self._k = _int_array(self.k)
        self.stream = stream

    def _head(self):
        return (self._arr, self.n, self._k)

    def _geom(self):
        return (self.B, self.V_local, self.rank, self.n_ranks, self.dt)

    def _ws(self):
        return (_ptr(self.workspace), self.workspace.numel(), _stream(self.stream))

    def stats(self):
        _check(self.lib.polyspec_sharded_chain_stats(*self._head(), *self._geom(), self.temperature, _ptr(self.stats_record),
                                                     _ptr(self.device_status), *self._ws()), "polyspec_sharded_chain_stats")
        return self.stats_record

    def gather(self, level):
        _check(self.lib.polyspec_sharded_chain_gather(*self._head(), level, _ptr(self.block_tokens), _ptr(self.block_len), *self._geom(),
                                                      _ptr(self.gather_record), *self._ws()), "polyspec_sharded_chain_gather")
        return self.gather_record

    def decide(self, level, stats_records, gather_records):
        _dev_check(stats_records, gather_records)
        if stats_records.numel() != self.n_ranks * self.stats_bytes or gather_records.numel() != self.n_ranks * self.gather_bytes:
            raise ValueError("need every rank's records, in rank order")
        _check(self.lib.polyspec_sharded_chain_decide(*self._head(), level, _ptr(self.block_tokens), _ptr(self.block_len), _ptr(self.uniforms),
                                                      *self._geom(), self.temperature, _ptr(stats_records), _ptr(gather_records),
                                                      _ptr(self.out["accepted_len"]), _ptr(self.out["block_len"]), _ptr(self.mass_record),
                                                      _ptr(self.device_status), *self._ws()), "polyspec_sharded_chain_decide")
        return self.mass_record

    def pick(self, level, mass_records):
        _dev_check(mass_records)
        if mass_records.numel() != self.n_ranks * self.mass_bytes:
            raise ValueError("need every rank's mass record, in rank order")
        _check(self.lib.polyspec_sharded_chain_pick(*self._head(), level, _ptr(self.uniforms), *self._geom(), self.temperature,
                                                    _ptr(mass_records), _ptr(self.next_token), _ptr(self.device_status), *self._ws()),
               "polyspec_sharded_chain_pick")
        return self.next_token

    def handoff(self, level, token):
        _dev_check(token)
        _check(self.lib.polyspec_sharded_chain_handoff(self.n, self._k, level, self.B, _ptr(self.out["accepted_len"]), _ptr(token),
                                                       _ptr(self.block_tokens), _ptr(self.block_len), _ptr(self.out["out_tokens"]),
                                                       _ptr(self.out["out_len"]), _stream(self.stream)), "polyspec_sharded_chain_handoff")
