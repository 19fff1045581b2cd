"""Staged verification with a threshold (Section 3.3, "Staged Verification"; Algorithm 1) as a host loop
around ``polyspec_verify_level``, for one sequence and three models on position-indexed logits.

Algorithm 1: M_3 drafts K tokens, M_2 verifies them, and what M_2 lets through is accumulated; once at
least ``mu`` tokens have accumulated, M_1 verifies the accumulated block in one pass, the accepted part
is committed and t advances.  Here each M_2 round contributes its whole emitted stream (accepted prefix
plus the replacement or bonus token), which is distributed as M_2's own samples, so that M_1 can verify
the accumulated block against q = M_2's rows and the committed text keeps M_1's distribution; a round
therefore always adds at least one token.  Accumulation also stops when another round could overflow the
largest block a level may verify.

The loop needs fresh logits after every round, which in a real system are model forwards; with synthetic
logits indexed by position (row i of every model scores position i, whatever the tokens before it) the
rows are simply slices, so the whole schedule can be run and measured: tokens committed per M_1 call as a
function of mu.  All verification arithmetic happens in the backend's ``level`` call (the CUDA library
through ``GpuLevel``); this module only slices, counts and appends.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List

import torch

MAX_BLOCK = 32          # POLYSPEC_MAX_K


class GpuLevel:
    """Backend that runs one sequence's level on the GPU through polyspec_verify_level."""

    def __init__(self, temperature: float):
        from . import binding
        self.binding = binding
        self.temperature = float(temperature)

    def level(self, rows_p: torch.Tensor, rows_q: torch.Tensor, tokens: torch.Tensor, uniforms: torch.Tensor):
        """rows_p [m+1, V], rows_q [m, V], tokens [m] int32, uniforms [m+1] float32 (device) -> (accepted, next)."""
        out = self.binding.polyspec_verify_level(rows_p.unsqueeze(0), rows_q.unsqueeze(0), tokens.unsqueeze(0),
                                                 uniforms.unsqueeze(0), self.temperature)
        res = torch.stack([out["accepted_len"][0], out["next_token"][0], out["device_status"][0]]).tolist()   # one sync
        if res[2] != 0 or res[0] < 0:
            raise RuntimeError(f"polyspec_verify_level reported device status {res[2]}")
        return int(res[0]), int(res[1])


@dataclass
class StagedResult:
    committed: List[int] = field(default_factory=list)      # the text M_1 committed, in order
    m1_calls: int = 0
    m2_calls: int = 0
    per_cycle: List[int] = field(default_factory=list)      # tokens committed by each M_1 call
    presented: List[int] = field(default_factory=list)      # block length presented to each M_1 call

    @property
    def tokens_per_m1_call(self) -> float:
        return len(self.committed) / max(self.m1_calls, 1)


def staged_decode(backend, M1: torch.Tensor, M2: torch.Tensor, M3: torch.Tensor, drafts: torch.Tensor,
                  u2: torch.Tensor, u1: torch.Tensor, K: int, mu: int, n_tokens: int) -> StagedResult:
    """Run Algorithm 1's schedule from position 0 until ``n_tokens`` are committed.

    M1, M2, M3   [N, V] logits by position (one sequence)
    drafts       [N] int32: the token M_3 proposes at each position
    u2           [rounds, K+1] uniforms of the M_2 rounds (row r for the r-th round overall)
    u1           [cycles, MAX_BLOCK+1] uniforms of the M_1 calls (slots 0..m-1 accept tests, slot MAX_BLOCK sampling)
    """
    if not (1 <= K <= MAX_BLOCK - 1 and 1 <= mu <= MAX_BLOCK):
        raise ValueError("need 1 <= K < 32 and 1 <= mu <= 32")
    res = StagedResult()
    t = 0
    N = M1.shape[0]
    while len(res.committed) < n_tokens:
        acc: List[int] = []
        # accumulate M_2-verified streams until the threshold (or until another round might not fit)
        while len(acc) < mu and len(acc) + K + 1 <= MAX_BLOCK:
            s = t + len(acc)
            if s + K + 1 > N or res.m2_calls >= u2.shape[0]:
                raise ValueError("ran out of positions or uniforms")
            a2, nxt = backend.level(M2[s:s + K + 1], M3[s:s + K], drafts[s:s + K], u2[res.m2_calls])
            res.m2_calls += 1
            acc.extend(int(x) for x in drafts[s:s + a2].tolist())
            acc.append(nxt)
        m = len(acc)
        if res.m1_calls >= u1.shape[0]:
            raise ValueError("ran out of uniforms")
        u = torch.cat([u1[res.m1_calls, :m], u1[res.m1_calls, MAX_BLOCK:MAX_BLOCK + 1]])
        block = torch.tensor(acc, dtype=torch.int32, device=M1.device)
        a1, nxt1 = backend.level(M1[t:t + m + 1], M2[t:t + m], block, u)
        res.m1_calls += 1
        res.presented.append(m)
        res.per_cycle.append(a1 + 1)
        res.committed.extend(acc[:a1])
        res.committed.append(nxt1)
        t += a1 + 1
    return res
