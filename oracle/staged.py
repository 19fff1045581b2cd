"""Staged verification with a threshold, for one sequence -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

Section 3.3 ("Staged Verification") and Algorithm 1, three models: M_3 drafts K tokens, M_2 verifies
them, what M_2 lets through is appended to `accepted` and counted in `cnt`; once cnt >= mu, M_1 verifies
the accumulated block in one pass, the verified part is committed, t advances, `accepted` and `cnt` are
reset.  The steps below are Algorithm 1's, in its order and with its names; each level call is the
oracle's own `verify_level` (the rule of Algorithm 1's Verify / VerifyBlock / SampleOne).

Readings, where the listing is silent or cannot be taken literally:
  - A round of M_2 hands on its whole emitted stream: the accepted prefix AND the token that replaces the
    first rejected draft (or follows a fully accepted block).  That stream is distributed as M_2's own
    samples, which is what lets M_1 verify it against q = M_2's rows and keeps M_1's distribution in the
    committed text; it also means every round adds at least one token, so the loop always terminates
    (the listing as printed appends accepted drafts only and would spin on a round that accepts nothing).
  - VerifyBlock is prefix acceptance with a replacement / bonus token, as everywhere in this oracle.
  - A level verifies at most `max_block` tokens, so accumulation also stops when one more round might
    not fit (len(accepted) + K + 1 > max_block).
  - Logits are indexed by position: row i of every model scores position i whatever the tokens before it
    (synthetic stand-in for the model forwards of the listing), and drafts[i] is M_3's proposal there.

Uniforms: u2[r] (K + 1 floats) serves the r-th M_2 round overall; u1[c] (max_block + 1 floats) the c-th
M_1 pass: slots 0..m-1 its accept tests, slot max_block its sampling uniform.

Pinned (tests/test_oracle_staged.py) by exact enumeration on tiny vocabularies: every branch of every
round and pass, with exact weights, must reproduce what the enumeration expects, and the law of the
committed prefix must equal the product of M_1's rows.
"""
from __future__ import annotations

import numpy as np

from . import oracle as _level

MAX_BLOCK = 32


def staged_decode(M1, M2, M3, drafts, u2, u1, K, mu, n_tokens, temperature, max_block=MAX_BLOCK):
    """Algorithm 1 from t = 0 until at least n_tokens are committed.

    M1, M2, M3  [N, V] logits by position (numpy float32/float64 or CPU torch tensors)
    drafts      [N] int32
    u2          [rounds, K+1] float32, u1 [cycles, max_block+1] float32
    Returns a dict: committed (list), m1_calls, m2_calls, presented (block length of each M_1 pass),
    per_cycle (tokens committed by each M_1 pass).
    """
    drafts = np.ascontiguousarray(drafts, dtype=np.int32)
    u2 = np.ascontiguousarray(u2, dtype=np.float32)
    u1 = np.ascontiguousarray(u1, dtype=np.float32)
    N = M1.shape[0]
    t = 0
    committed, presented, per_cycle = [], [], []
    m1_calls = m2_calls = 0
    while len(committed) < n_tokens:
        accepted = []
        cnt = 0
        # draft with M_3 and verify with M_2 until the threshold is reached
        while cnt < mu and cnt + K + 1 <= max_block:
            s = t + cnt
            if s + K + 1 > N or m2_calls >= u2.shape[0]:
                raise ValueError("ran out of positions or uniforms")
            x = drafts[s:s + K]
            out = _level.verify_level(M2[s:s + K + 1][None], M3[s:s + K][None], x[None], u2[m2_calls][None], temperature)
            if out["status"][0] != 0:
                raise ValueError("unusable input")
            m2_calls += 1
            a2 = int(out["accepted_len"][0])
            for i in range(a2):
                accepted.append(int(x[i]))
            accepted.append(int(out["next_token"][0]))
            cnt = len(accepted)
        # threshold reached: M_1 verifies the accumulated block against q = M_2's rows
        if m1_calls >= u1.shape[0] or t + cnt + 1 > N:
            raise ValueError("ran out of positions or uniforms")
        u = np.concatenate([u1[m1_calls, :cnt], u1[m1_calls, max_block:max_block + 1]])
        out = _level.verify_level(M1[t:t + cnt + 1][None], M2[t:t + cnt][None], np.array([accepted], np.int32), u[None], temperature)
        if out["status"][0] != 0:
            raise ValueError("unusable input")
        m1_calls += 1
        a1 = int(out["accepted_len"][0])
        presented.append(cnt)
        per_cycle.append(a1 + 1)
        committed.extend(accepted[:a1])
        committed.append(int(out["next_token"][0]))
        t += a1 + 1
    return {"committed": committed, "m1_calls": m1_calls, "m2_calls": m2_calls, "presented": presented, "per_cycle": per_cycle}
