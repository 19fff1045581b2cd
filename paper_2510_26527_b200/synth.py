"""Seeded synthetic inputs for the verification step.

This module only *makes inputs*: logits (or hidden states and LM-head weights),
draft tokens and the uniforms a caller would supply.  It holds none of the
verification arithmetic, imports neither the CUDA binding nor the CPU oracle,
and serves both.  The shapes follow LLaMA2 / LLaMA3 / Qwen2 vocabularies
(32000 / 128256 / 152064) and the block lengths of the benchmark configurations;
the values are Gaussian logits with per-level Gaussian noise, standing in for
real model outputs, which are not available offline.

Uniforms come from Philox4x32-10 (Salmon et al., "Parallel random numbers: as
easy as 1, 2, 3"): key = (seed low word, seed high word), counter =
(level, sequence, slot, 0), first output word w, u = ((w >> 8) + 0.5) * 2^-24,
which lies strictly inside (0, 1) and is exact in float32.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import Optional, Sequence

import numpy as np
import torch

_PHILOX_M0 = np.uint64(0xD2511F53)
_PHILOX_M1 = np.uint64(0xCD9E8D57)
_PHILOX_W0 = 0x9E3779B9
_PHILOX_W1 = 0xBB67AE85
_MASK32 = np.uint64(0xFFFFFFFF)


def philox4x32_10(counter: np.ndarray, key: Sequence[int]) -> np.ndarray:
    """Philox4x32 with 10 rounds.  counter: uint32 [..., 4]; key: two 32-bit words."""
    c = np.asarray(counter, dtype=np.uint64) & _MASK32
    c0, c1, c2, c3 = (c[..., i].copy() for i in range(4))
    k0, k1 = int(key[0]) & 0xFFFFFFFF, int(key[1]) & 0xFFFFFFFF
    for r in range(10):
        p0 = _PHILOX_M0 * c0
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK32
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK32
        c0, c1, c2, c3 = (hi1 ^ c1 ^ np.uint64(k0)), lo1, (hi0 ^ c3 ^ np.uint64(k1)), lo0
        k0 = (k0 + _PHILOX_W0) & 0xFFFFFFFF
        k1 = (k1 + _PHILOX_W1) & 0xFFFFFFFF
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def philox_uniforms(seed: int, levels: int, batch: int, slots: int, batch_offset: int = 0) -> np.ndarray:
    """float32 [levels, batch, slots] of uniforms in (0, 1), one Philox call per entry."""
    l, b, j = np.meshgrid(np.arange(levels, dtype=np.uint64),
                          np.arange(batch_offset, batch_offset + batch, dtype=np.uint64),
                          np.arange(slots, dtype=np.uint64), indexing="ij")
    ctr = np.stack([l, b, j, np.zeros_like(l)], axis=-1)
    w = philox4x32_10(ctr, (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF))[..., 0]
    u = ((w >> np.uint32(8)).astype(np.float64) + 0.5) * (2.0 ** -24)
    return u.astype(np.float32)


@dataclass(frozen=True)
class ChainSpec:
    """A logits-path workload: n models, levels l = 0 (M_1's) .. n-2 (the bottom)."""
    name: str
    n_models: int
    B: int
    V: int
    dtype: torch.dtype
    k: tuple                      # k[l] = largest block level l verifies; k[-1] = draft length
    temperature: float
    base_std: float
    sigmas: tuple                 # noise std of models 2..n
    cumulative: bool              # True: M_{i+1} = M_i + noise; False: M_{i+1} = M_1 + noise
    boost_frac: float = 0.0       # fraction of entries per row raised by boost_amount
    boost_amount: float = 0.0

    @property
    def rows(self) -> tuple:
        L = self.n_models - 1
        return tuple(self.k[i] + 1 for i in range(L)) + (self.k[L - 1],)

    @property
    def kmax(self) -> int:
        return max(self.k)

    def logits_bytes(self) -> int:
        elem = 4 if self.dtype == torch.float32 else 2
        return sum(self.rows) * self.B * self.V * elem


def config(name: str, sigma: Optional[float] = None) -> ChainSpec:
    """The benchmark's logits-path configurations (config 4 is the fused path, see FusedSpec)."""
    if name == "cfg1":   # two-level, batch 1, k=4, V=32000, fp32
        return ChainSpec("cfg1", 2, 1, 32000, torch.float32, (4,), 1.0, 3.0, (1.0,), False)
    if name == "cfg2":   # three-level, batch 1, V=32000, bf16; level 1 has no cap below 9
        return ChainSpec("cfg2", 3, 1, 32000, torch.bfloat16, (9, 8), 1.0, 3.0, (0.5, 1.5), False)
    if name == "cfg3":   # three-level, batch 64, V=128256, bf16, peaked rows, T=0.7
        return ChainSpec("cfg3", 3, 64, 128256, torch.bfloat16, (6, 6), 0.7, 4.0, (0.75, 2.0), False,
                         boost_frac=0.01, boost_amount=8.0)
    if name == "cfg5":   # four-level, batch 256, V=152064, bf16, k=(10,6,4) bottom-up
        s = 1.0 if sigma is None else float(sigma)
        return ChainSpec("cfg5", 4, 256, 152064, torch.bfloat16, (4, 6, 10), 1.0, 3.0, (s, s, s), True)
    raise KeyError(name)


CFG5_SIGMAS = (0.25, 0.5, 1.0, 2.0, 4.0)


def scaled(spec: ChainSpec, B: Optional[int] = None, V: Optional[int] = None) -> ChainSpec:
    """The same recipe at a reduced batch and/or vocabulary (for tests the oracle finishes quickly)."""
    return replace(spec, B=spec.B if B is None else B, V=spec.V if V is None else V)


def make_chain(spec: ChainSpec, seed: int, device="cpu", batch_offset: int = 0) -> dict:
    """Logits of every model, the bottom draft tokens and the uniforms for one call.

    Logits are drawn in float32 and rounded once to ``spec.dtype``; draft tokens are
    sampled from the softmax of the *stored* bottom-model logits at the call's
    temperature.  ``batch_offset`` shifts the Philox sequence index so that ranks of a
    data-parallel run draw distinct uniforms.
    """
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(int(seed) * 1000003 + batch_offset)
    rows = spec.rows
    R = max(rows)
    B, V = spec.B, spec.V
    base = torch.randn((B, R, V), generator=g, device=dev, dtype=torch.float32) * spec.base_std
    if spec.boost_frac > 0.0:
        cnt = max(1, int(round(spec.boost_frac * V)))
        idx = torch.rand((B, R, V), generator=g, device=dev).topk(cnt, dim=-1).indices
        base.scatter_add_(-1, idx, torch.full(idx.shape, spec.boost_amount, device=dev, dtype=torch.float32))
        del idx
    models = [base[:, :rows[0]].to(spec.dtype).contiguous()]
    prev = base
    for i in range(1, spec.n_models):
        noise = torch.randn((B, R, V), generator=g, device=dev, dtype=torch.float32) * spec.sigmas[i - 1]
        cur = (prev if spec.cumulative else base) + noise
        del noise
        models.append(cur[:, :rows[i]].to(spec.dtype).contiguous())
        prev = cur
    del prev, base
    probs = torch.softmax(models[-1].to(torch.float32) / spec.temperature, dim=-1)
    kb = spec.k[-1]
    draft = torch.multinomial(probs.reshape(B * kb, V), 1, generator=g).reshape(B, kb).to(torch.int32)
    del probs
    L = spec.n_models - 1
    u = torch.from_numpy(philox_uniforms(seed, L, B, spec.kmax + 1, batch_offset)).to(dev)
    return {"spec": spec, "models": models, "k": list(spec.k), "draft_tokens": draft.contiguous(),
            "uniforms": u.contiguous(), "temperature": spec.temperature}


@dataclass(frozen=True)
class FusedSpec:
    """The fused LM-head workload: hidden states and LM-head weights instead of logits."""
    name: str = "cfg4"
    B: int = 32
    k: int = 8
    V: int = 32000
    d_p: int = 4096
    d_q: int = 2048
    temperature: float = 1.0
    w_std: float = 0.02
    logit_std: float = 3.0
    shared_frac: float = 0.9      # share of the target logits' variance carried by the first d_q features

    @property
    def rows_q(self) -> int:
        return self.k + 1

    def weight_bytes(self) -> int:
        return 2 * self.V * (self.d_p + self.d_q)

    def flops(self) -> int:
        return 2 * self.B * (self.k + 1) * self.V * (self.d_p + self.d_q)


def make_fused(spec: FusedSpec, seed: int, device="cpu") -> dict:
    """Hidden states / weights such that target logits have std ~ logit_std and the draft tracks them.

    W_p ~ N(0, w_std^2).  The draft model sees the first d_q features: W_q = W_p[:, :d_q] and
    hidden_q = hidden_p[..., :d_q] / sqrt(shared_frac), so its logits are a rescaled partial sum
    of the target's (the remaining d_p - d_q features carry 1 - shared_frac of the variance and
    act as the draft's error).  Draft tokens are sampled from the draft softmax computed with a
    float32 matmul of the stored bf16 values.
    """
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(int(seed) * 1000003 + 4)
    B, k, V, dp, dq = spec.B, spec.k, spec.V, spec.d_p, spec.d_q
    assert dq < dp
    W_p = (torch.randn((V, dp), generator=g, device=dev, dtype=torch.float32) * spec.w_std).to(torch.bfloat16)
    s1 = math.sqrt(spec.shared_frac) * spec.logit_std / (spec.w_std * math.sqrt(dq))
    s2 = math.sqrt(1.0 - spec.shared_frac) * spec.logit_std / (spec.w_std * math.sqrt(dp - dq))
    h = torch.randn((B, k + 1, dp), generator=g, device=dev, dtype=torch.float32)
    h[..., :dq] *= s1
    h[..., dq:] *= s2
    hidden_p = h.to(torch.bfloat16).contiguous()
    hidden_q = (h[..., :dq] / math.sqrt(spec.shared_frac)).to(torch.bfloat16).contiguous()
    W_q = W_p[:, :dq].contiguous()
    lq = torch.matmul(hidden_q[:, :k].to(torch.float32), W_q.to(torch.float32).t())
    probs = torch.softmax(lq / spec.temperature, dim=-1)
    draft = torch.multinomial(probs.reshape(B * k, V), 1, generator=g).reshape(B, k).to(torch.int32)
    u = torch.from_numpy(philox_uniforms(seed, 1, B, k + 1)[0]).to(dev)
    return {"spec": spec, "hidden_p": hidden_p, "W_p": W_p.contiguous(), "hidden_q": hidden_q, "W_q": W_q,
            "draft_tokens": draft.contiguous(), "uniforms": u.contiguous(), "temperature": spec.temperature}
