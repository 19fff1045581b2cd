"""Pins of the oracle's staged schedule (Section 3.3 "Staged Verification", Algorithm 1; oracle/staged.py).

Exact enumeration on a tiny vocabulary.  The enumeration below is written on its own from probability tables
(scipy's softmax): it walks every branch of every M_2 round and every M_1 pass of the schedule with exact
weights -- each draft token weighted by M_3's probability the first time its position is drafted, each accept
uniform at the midpoint of its accept or reject region, each sampling uniform at the midpoint of a token's CDF
interval -- and says what the schedule must do on that branch.  Driving the oracle with those drafts and
uniforms must reproduce it (committed text, blocks presented to M_1, tokens per pass, call counts), and the law of
the committed prefix must be the product of M_1's rows: the schedule is lossless although several M_2 rounds are
accumulated before M_1 looks, and although a position's draft is met again after a rejection before it.
"""
import numpy as np
import pytest

from oracle import staged as ostaged
from tests import helpers as H

MAXB = ostaged.MAX_BLOCK


def enumerate_schedule(P1, P2, Q3, K, mu, n_tokens, V, max_block=MAXB):
    """Yield (weight, drafts {position: token}, u2 rows, u1 rows, committed, presented, per_cycle) over all branches."""

    def cycle(t, committed, presented, per_cycle, drafts, u2_rows, u1_rows, weight):
        if len(committed) >= n_tokens:
            yield weight, drafts, u2_rows, u1_rows, committed, presented, per_cycle
            return
        yield from accumulate(t, [], committed, presented, per_cycle, drafts, u2_rows, u1_rows, weight)

    def accumulate(t, acc, committed, presented, per_cycle, drafts, u2_rows, u1_rows, weight):
        if len(acc) >= mu or len(acc) + K + 1 > max_block:
            m = len(acc)
            _, branches = H.level_branches(P1[t:t + m + 1], P2[t:t + m], acc, m)
            for a1, v, w, ua, us in branches:
                row = [0.5] * (max_block + 1)
                row[:m] = ua
                row[max_block] = us
                yield from cycle(t + a1 + 1, committed + acc[:a1] + [v], presented + [m], per_cycle + [a1 + 1],
                                 drafts, u2_rows, u1_rows + [row], weight * w)
            return
        s = t + len(acc)
        fresh = [i for i in range(s, s + K) if i not in drafts]

        def assign(idx, d, w):
            if idx == len(fresh):
                yield d, w
                return
            for v in range(V):
                yield from assign(idx + 1, {**d, fresh[idx]: v}, w * Q3[fresh[idx], v])

        for d, wd in assign(0, drafts, 1.0):
            stream = [d[i] for i in range(s, s + K)]
            _, branches = H.level_branches(P2[s:s + K + 1], Q3[s:s + K], stream, K)
            for a2, v, w, ua, us in branches:
                yield from accumulate(t, acc + stream[:a2] + [v], committed, presented, per_cycle, d,
                                      u2_rows + [list(ua) + [us]], u1_rows, weight * wd * w)

    yield from cycle(0, [], [], [], {}, [], [], 1.0)


@pytest.mark.parametrize("V,K,mu,n_tokens,T,seed", [(2, 1, 2, 2, 1.0, 0), (2, 2, 2, 2, 0.8, 1), (3, 1, 1, 2, 1.0, 2),
                                                     (2, 2, 3, 1, 1.0, 3), (3, 2, 2, 1, 1.3, 4), (2, 1, 3, 3, 1.0, 5)])
def test_schedule_by_exact_enumeration(V, K, mu, n_tokens, T, seed):
    r = np.random.default_rng(300 + seed)
    N = n_tokens + mu + 2 * K + 3
    M1 = r.normal(0, 1.2, (N, V))
    M2 = M1 + r.normal(0, 0.8, (N, V))
    M3 = M1 + r.normal(0, 1.1, (N, V))
    P1, P2, Q3 = H.prob_tables([M1, M2, M3], T)
    total, leaves = 0.0, 0
    prefix = {}                                   # first n_tokens committed tokens -> mass
    for weight, drafts, u2_rows, u1_rows, committed, presented, per_cycle in enumerate_schedule(P1, P2, Q3, K, mu, n_tokens, V):
        d = np.zeros(N, np.int32)
        for pos, tok in drafts.items():
            d[pos] = tok
        u2 = np.array(u2_rows + [[0.5] * (K + 1)], np.float32)
        u1 = np.array(u1_rows + [[0.5] * (MAXB + 1)], np.float32)
        got = ostaged.staged_decode(M1, M2, M3, d, u2, u1, K, mu, n_tokens, T)
        assert got["committed"] == committed, (drafts, u2_rows, u1_rows, got, committed)
        assert got["presented"] == presented and got["per_cycle"] == per_cycle
        assert got["m2_calls"] == len(u2_rows) and got["m1_calls"] == len(u1_rows)
        # bookkeeping the listing fixes: a pass sees at least min(mu, ...) tokens and commits at most one more than it saw
        for m, c in zip(presented, per_cycle):
            assert m >= min(mu, MAXB - K) and 1 <= c <= m + 1
        key = tuple(committed[:n_tokens])
        prefix[key] = prefix.get(key, 0.0) + weight
        total += weight
        leaves += 1
    assert abs(total - 1.0) < 1e-12, total
    assert leaves > 20
    # the committed prefix follows M_1's rows, position by position
    for y, mass in prefix.items():
        expect = np.prod([P1[i, y[i]] for i in range(n_tokens)])
        assert abs(mass - expect) < 1e-12, (y, mass, expect)
    assert abs(sum(prefix.values()) - 1.0) < 1e-12


def test_schedule_reduces_to_the_chain_when_one_round_fills_the_block():
    """mu = 1: every cycle is one M_2 round followed by the M_1 pass on its stream, i.e. one call of the three-model
    chain with no cap at M_1's level; the first cycle must equal the chain oracle on the same rows and uniforms."""
    from oracle import oracle as orc
    from paper_2510_26527_b200 import synth
    V, K, T = 50, 4, 0.9
    r = np.random.default_rng(9)
    N = 40
    M1 = r.normal(0, 2.0, (N, V)).astype(np.float32)
    M2 = (M1 + r.normal(0, 0.6, (N, V))).astype(np.float32)
    M3 = (M1 + r.normal(0, 1.2, (N, V))).astype(np.float32)
    Q3 = H.prob_tables([M3], T)[0]
    for trial in range(30):
        drafts = np.array([r.choice(V, p=Q3[i]) for i in range(N)], np.int32)
        u2 = synth.philox_uniforms(50 + trial, 1, 8, K + 1)[0]
        u1 = synth.philox_uniforms(90 + trial, 1, 8, MAXB + 1)[0]
        got = ostaged.staged_decode(M1, M2, M3, drafts, u2, u1, K, 1, 1, T)
        kk = [K + 1, K]
        U = np.zeros((2, 1, K + 2), np.float32)
        U[1, 0, :K] = u2[0, :K]
        U[1, 0, K + 1] = u2[0, K]
        U[0, 0, :K + 1] = u1[0, :K + 1]
        U[0, 0, K + 1] = u1[0, MAXB]
        ch = orc.verify_chain([M1[None, :K + 2], M2[None, :K + 1], M3[None, :K]], kk, drafts[None, :K], U, T)
        n = int(ch["out_len"][0, 0])
        assert got["committed"] == ch["out_tokens"][0, 0, :n].tolist()
        assert got["presented"] == [int(ch["block_len"][0, 0])] and got["m2_calls"] == 1
