"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

  (a) exact enumeration on tiny vocabularies: the emitted stream keeps the verifier's law
      (the paper's claim that the output distribution of the target is preserved: abstract,
      Sections 1 and 5), single level and chains of 3 and 4 models;
  (b) p == q accepts every draft;  (c) disjoint supports reject at position 1 and the
      residual is p;  (d) the residual mass is 1 - sum min(p, q) and the normalised residual
      sums to 1;  (e) the mean acceptance length matches sum_j prod alpha_i (Eq. 1; the
      constant-alpha case is the capped-geometric mean in the proof of Theorem 3.3);
  library routines: scipy softmax, numpy cumsum + searchsorted.
"""
import numpy as np
import pytest
import torch
from scipy.special import softmax as sp_softmax

from tests import helpers as H
from paper_2510_26527_b200 import synth


def _rng(seed):
    return np.random.default_rng(seed)


# ---------------------------------------------------------------- softmax
@pytest.mark.parametrize("T", [0.3, 0.7, 1.0, 2.5])
def test_softmax_matches_library_routine(oracle, T):
    z = _rng(1).normal(0, 3, size=1000).astype(np.float32)
    z[[3, 500]] = -np.inf
    P = oracle.softmax_row(z, T)
    ref = sp_softmax(z.astype(np.float64) / T)
    np.testing.assert_allclose(P, ref, rtol=1e-12, atol=0)
    assert P[3] == 0.0 and abs(P.sum() - 1.0) < 1e-12


def test_softmax_dtypes_and_limits(oracle):
    z = torch.randn(777, generator=torch.Generator().manual_seed(2)) * 3
    zb = z.to(torch.bfloat16)
    np.testing.assert_allclose(oracle.softmax_row(zb, 1.0), sp_softmax(zb.double().numpy()), rtol=1e-12)
    np.testing.assert_allclose(oracle.softmax_row(zb.view(torch.int16).numpy().view(np.uint16), 1.0),
                               sp_softmax(zb.double().numpy()), rtol=1e-12)
    np.testing.assert_allclose(oracle.softmax_row(z.double(), 0.5), sp_softmax(z.double().numpy() / 0.5), rtol=1e-12)
    # very high temperature flattens the row
    np.testing.assert_allclose(oracle.softmax_row(z, 1e9), np.full(777, 1 / 777), rtol=1e-6)
    # shifting every logit leaves the distribution unchanged
    np.testing.assert_allclose(oracle.softmax_row(z.double() + 100.0, 1.0), oracle.softmax_row(z.double(), 1.0), rtol=1e-9)


def test_softmax_rejects_unusable_rows(oracle):
    z = np.zeros(8, np.float32)
    z[2] = np.nan
    with pytest.raises(ValueError):
        oracle.softmax_row(z, 1.0)
    with pytest.raises(ValueError):
        oracle.softmax_row(np.full(8, -np.inf, np.float32), 1.0)
    z[2] = np.inf
    with pytest.raises(ValueError):
        oracle.softmax_row(z, 1.0)


# ---------------------------------------------------------------- (b) p == q
def test_identical_models_accept_every_draft(oracle):
    B, k, V = 64, 7, 50
    r = _rng(3)
    lp = r.normal(0, 3, (B, k + 1, V)).astype(np.float32)
    lq = lp[:, :k].copy()
    tok = r.integers(0, V, (B, k)).astype(np.int32)
    u = synth.philox_uniforms(3, 1, B, k + 1)[0]
    u[:, 0] = np.float32(1.0 - 2.0 ** -25)       # the largest uniform the generator can produce
    u[:, 1] = np.float32(2.0 ** -25)             # and the smallest
    out = oracle.verify_level(lp, lq, tok, u, 1.0)
    assert (out["accepted_len"] == k).all() and (out["status"] == 0).all()
    # the bonus token is the inverse CDF of row k at the sampling uniform
    for b in range(B):
        cdf = np.cumsum(sp_softmax(lp[b, k].astype(np.float64)))
        assert out["next_token"][b] == np.searchsorted(cdf, float(u[b, k]), side="right")


# ---------------------------------------------------------------- (c) disjoint supports
def test_disjoint_supports_reject_at_first_position(oracle):
    B, k, V = 32, 4, 40
    r = _rng(4)
    lp = r.normal(0, 2, (B, k + 1, V)).astype(np.float32)
    lq = r.normal(0, 2, (B, k, V)).astype(np.float32)
    lp[:, :, : V // 2] = -np.inf          # target mass on the upper half only
    lq[:, :, V // 2:] = -np.inf           # draft mass on the lower half only
    tok = r.integers(0, V // 2, (B, k)).astype(np.int32)
    u = synth.philox_uniforms(4, 1, B, k + 1)[0]
    out = oracle.verify_level(lp, lq, tok, u, 1.0)
    assert (out["accepted_len"] == 0).all()
    np.testing.assert_allclose(out["sample_info"][:, 1], 1.0, rtol=1e-12)     # residual mass = 1 (d)
    for b in range(B):                    # residual == p: plain inverse CDF of p's first row
        cdf = np.cumsum(sp_softmax(lp[b, 0].astype(np.float64)))
        assert out["next_token"][b] == np.searchsorted(cdf, float(u[b, k]) * cdf[-1], side="right")
        assert out["next_token"][b] >= V // 2


# ---------------------------------------------------------------- (d) residual + inverse CDF
def test_residual_mass_and_inverse_cdf_match_numpy(oracle):
    B, k, V = 200, 3, 97
    r = _rng(5)
    lp = r.normal(0, 3, (B, k + 1, V)).astype(np.float32)
    lq = (lp[:, :k] + r.normal(0, 1.5, (B, k, V))).astype(np.float32)
    T = 0.8
    Q = sp_softmax(lq.astype(np.float64) / T, axis=-1)
    P = sp_softmax(lp.astype(np.float64) / T, axis=-1)
    tok = np.stack([[r.choice(V, p=Q[b, j]) for j in range(k)] for b in range(B)]).astype(np.int32)
    u = synth.philox_uniforms(5, 1, B, k + 1)[0]
    out = oracle.verify_level(lp, lq, tok, u, T)
    seen_reject = seen_bonus = 0
    for b in range(B):
        # accepted length by the definition, position by position
        a = 0
        while a < k and float(u[b, a]) * Q[b, a, tok[b, a]] <= P[b, a, tok[b, a]]:
            a += 1
        assert out["accepted_len"][b] == a
        if a < k:
            res = np.maximum(P[b, a] - Q[b, a], 0.0)
            alpha = np.minimum(P[b, a], Q[b, a]).sum()
            assert abs(out["sample_info"][b, 1] - (1.0 - alpha)) < 1e-12      # S = 1 - alpha
            assert abs((res / res.sum()).sum() - 1.0) < 1e-12
            cdf = np.cumsum(res)
            expect = np.searchsorted(cdf, float(u[b, k]) * cdf[-1], side="right")
            seen_reject += 1
        else:
            cdf = np.cumsum(P[b, k])
            expect = np.searchsorted(cdf, float(u[b, k]), side="right")
            seen_bonus += 1
        assert out["next_token"][b] == expect
        np.testing.assert_allclose(out["p_at"][b, : min(a + 1, k)], P[b, np.arange(min(a + 1, k)), tok[b, : min(a + 1, k)]], rtol=1e-12)
        np.testing.assert_allclose(out["q_at"][b, : min(a + 1, k)], Q[b, np.arange(min(a + 1, k)), tok[b, : min(a + 1, k)]], rtol=1e-12)
    assert seen_reject > 20 and seen_bonus > 5


def test_margins_and_neighbours(oracle):
    # a hand-made case: P = (0.5, 0, 0.25, 0.25), Q = uniform over 4; token 0 drafted.
    lp = np.log(np.array([[[0.5, 1e-300, 0.25, 0.25]] * 2], dtype=np.float64))
    lp[0, :, 1] = -np.inf
    lq = np.zeros((1, 1, 4), dtype=np.float64)
    tok = np.array([[1]], dtype=np.int32)                     # Q(1)=0.25, P(1)=0 -> always rejected
    u = np.array([[0.3, 0.6]], dtype=np.float32)
    out = oracle.verify_level(lp, lq, tok, u, 1.0)
    assert out["accepted_len"][0] == 0
    # residual = max(0, P-Q) = (0.25, 0, 0, 0) -> token 0 whatever the uniform
    assert out["next_token"][0] == 0 and abs(out["sample_info"][0, 1] - 0.25) < 1e-15
    assert abs(out["accept_margin"][0, 0] - 0.3) < 1e-7       # |u - min(1, 0/0.25)|
    # bonus row sampling: accept token 0 (P/Q = 2), then the bonus row P at u_s = 0.6 -> token 2
    tok = np.array([[0]], dtype=np.int32)
    out = oracle.verify_level(lp, lq, tok, u, 1.0)
    assert out["accepted_len"][0] == 1 and out["next_token"][0] == 2
    margin, total, prev, succ = out["sample_info"][0]
    assert abs(margin - 0.1) < 1e-7 and total == 1.0 and prev == 0 and succ == 3   # zero-mass token 1 is skipped


def test_block_len_and_bad_inputs(oracle):
    B, k, V = 6, 4, 16
    r = _rng(6)
    lp = r.normal(0, 1, (B, k + 1, V)).astype(np.float32)
    lq = lp[:, :k].copy()
    tok = r.integers(0, V, (B, k)).astype(np.int32)
    u = synth.philox_uniforms(6, 1, B, k + 1)[0]
    bl = np.array([0, 1, 2, 3, 4, 2], dtype=np.int32)
    out = oracle.verify_level(lp, lq, tok, u, 1.0, block_len=bl)
    assert (out["accepted_len"] == bl).all()            # p == q: everything presented is accepted
    for b in range(B):                                   # bonus comes from row block_len[b]
        cdf = np.cumsum(sp_softmax(lp[b, bl[b]].astype(np.float64)))
        assert out["next_token"][b] == np.searchsorted(cdf, float(u[b, k]), side="right")
    tok[1, 0] = V
    lp[2, 0, 3] = np.nan
    out = oracle.verify_level(lp, lq, tok, u, 1.0, block_len=bl)
    assert out["status"][1] == 3 and out["accepted_len"][1] == -1 and out["next_token"][1] == -1
    assert out["status"][2] == 1 and out["accepted_len"][2] == -1
    assert out["status"][0] == 0 and out["status"][3] == 0


# ---------------------------------------------------------------- (a) exact enumeration, single level
@pytest.mark.parametrize("V,k,T,seed", [(4, 2, 1.0, 0), (5, 3, 0.7, 1), (8, 2, 1.3, 2), (3, 3, 1.0, 3)])
def test_single_level_stream_law_by_enumeration(oracle, V, k, T, seed):
    r = _rng(100 + seed)
    lp = r.normal(0, 1.5, (k + 1, V))
    lq = lp[:k] + r.normal(0, 1.0, (k, V))
    P, Q = H.prob_tables([lp, lq], T)
    law = {}                                   # (i, prefix y_1..y_i) -> mass of "stream has >= i tokens and starts with y"
    total = 0.0
    exp_a = 0.0
    for weight, U, draft, trace in H.enumerate_chain([P, Q], [k], V):
        (_, m, a, stream), = trace
        out = oracle.verify_level(lp[None], lq[None], np.array([draft], np.int32), U.astype(np.float32), T)
        assert out["accepted_len"][0] == a and out["next_token"][0] == stream[-1], (draft, U, trace)
        total += weight
        exp_a += weight * a
        for i in range(1, len(stream) + 1):
            key = (i, tuple(stream[:i]))
            law[key] = law.get(key, 0.0) + weight
    assert abs(total - 1.0) < 1e-12
    # joint law: Pr[len >= i, first i tokens = y] = prod_{j<i} min(P_j, Q_j)(y_j) * P_i(y_i)
    for (i, y), mass in law.items():
        expect = P[i - 1, y[-1]]
        for j in range(i - 1):
            expect *= min(P[j, y[j]], Q[j, y[j]])
        assert abs(mass - expect) < 1e-12, (i, y, mass, expect)
    # first-token marginal is exactly the target's first row
    for v in range(V):
        assert abs(law.get((1, (v,)), 0.0) - P[0, v]) < 1e-12
    # Eq. 1: the expected acceptance length is sum_j prod alpha_i
    assert abs(exp_a - H.expected_accept_len_bottom(P, Q, k)) < 1e-12


def test_literal_all_or_nothing_reading_is_not_lossless():
    """Algorithm 1 as printed accepts the whole block or draws a fresh token from the target's first
    row.  On a 2-token vocabulary that reading changes the first token's law, which is why the
    oracle implements prefix acceptance with residual resampling instead."""
    P = np.array([[0.8, 0.2], [0.5, 0.5]])
    Q = np.array([[0.5, 0.5], [0.9, 0.1]])
    first = np.zeros(2)
    for x1 in range(2):
        for x2 in range(2):
            w = Q[0, x1] * Q[1, x2]
            acc = min(1, P[0, x1] / Q[0, x1]) * min(1, P[1, x2] / Q[1, x2])
            first[x1] += w * acc                 # block accepted: first token is the draft's
            first += w * (1 - acc) * P[0]        # otherwise SampleOne(v_1)
    assert abs(first.sum() - 1) < 1e-12 and np.abs(first - P[0]).max() > 1e-2


# ---------------------------------------------------------------- (a) exact enumeration, chains
@pytest.mark.parametrize("n,k,seed", [(3, (2, 2), 0), (3, (1, 2), 1), (3, (3, 2), 2), (4, (2, 2, 2), 3), (4, (1, 2, 3), 4)])
def test_chain_stream_law_by_enumeration(oracle, n, k, seed):
    V, T = 3, 1.0
    r = _rng(200 + seed)
    L = n - 1
    rows = [k[i] + 1 for i in range(L)] + [k[L - 1]]
    R = max(rows)
    base = r.normal(0, 1.2, (R, V))
    logits = [base[: rows[0]]]
    for i in range(1, n):
        logits.append((base + r.normal(0, 0.9, (R, V)))[: rows[i]])
    tables = H.prob_tables(logits, T)
    kmax = max(k)
    pos_mass = np.zeros((kmax + 2, V))
    len_mass = np.zeros(kmax + 2)
    exp_a = np.zeros(L)
    total = 0.0
    models = [np.ascontiguousarray(l[None]) for l in logits]
    for weight, U, draft, trace in H.enumerate_chain(tables, list(k), V):
        out = oracle.verify_chain(models, list(k), np.array([draft], np.int32), U.astype(np.float32)[:, None, :], T)
        for (l, m, a, stream) in trace:
            assert out["block_len"][l, 0] == m and out["accepted_len"][l, 0] == a
            assert out["out_len"][l, 0] == a + 1
            assert list(out["out_tokens"][l, 0, : a + 1]) == stream
            assert (out["out_tokens"][l, 0, a + 1:] == -1).all()
            exp_a[l] += weight * a
        total += weight
        final = trace[-1][3]
        for i, y in enumerate(final):
            pos_mass[i, y] += weight
            len_mass[i] += weight
    assert abs(total - 1.0) < 1e-12
    P1 = tables[0]
    for i in range(min(kmax + 1, P1.shape[0])):
        if len_mass[i] > 0:
            np.testing.assert_allclose(pos_mass[i] / len_mass[i], P1[i], atol=1e-12)
    assert abs(len_mass[0] - 1.0) < 1e-12      # a cycle always commits at least one token
    # closed forms: bottom level, and the level above it
    assert abs(exp_a[L - 1] - H.expected_accept_len_bottom(tables[L - 1], tables[L], k[L - 1])) < 1e-12
    assert abs(exp_a[L - 2] - H.expected_accept_len_second(tables[L - 2], tables[L - 1], tables[L], k[L - 2], k[L - 1])) < 1e-12


def test_upper_level_must_use_the_verifier_below_as_q():
    """With q taken from the bottom drafter at M_1's level the first token's law is wrong; with
    q = M_2's distribution it is exact.  A two-position, two-token example, k = (1, 1)."""
    P1 = np.array([0.7, 0.3]); P2 = np.array([0.4, 0.6]); Q3 = np.array([0.1, 0.9])
    # stream after level 2 (k=1): accepted draft or residual -> law is exactly P2
    s2 = np.zeros(2)
    for x in range(2):
        t = min(1, P2[x] / Q3[x])
        s2[x] += Q3[x] * t
        res = np.maximum(P2 - Q3, 0); res /= res.sum()
        s2 += Q3[x] * (1 - t) * res
    np.testing.assert_allclose(s2, P2, atol=1e-15)

    def first_token_law(q):
        out = np.zeros(2)
        for x in range(2):
            t = min(1, P1[x] / q[x])
            out[x] += s2[x] * t
            res = np.maximum(P1 - q, 0); res /= res.sum()
            out += s2[x] * (1 - t) * res
        return out
    np.testing.assert_allclose(first_token_law(P2), P1, atol=1e-15)
    assert np.abs(first_token_law(Q3) - P1).max() > 1e-2


# ---------------------------------------------------------------- (e) acceptance-length statistics
def test_mean_acceptance_length_matches_closed_form(oracle):
    B, k, V, T = 3000, 6, 48, 1.0
    r = _rng(7)
    lp = r.normal(0, 3, (B, k + 1, V)).astype(np.float32)
    lq = (lp[:, :k] + r.normal(0, 1.0, (B, k, V))).astype(np.float32)
    P, Q = H.prob_tables([lp, lq], T)
    cdf = np.cumsum(Q, axis=-1)
    tok = (r.random((B, k, 1)) * cdf[..., -1:] > cdf).sum(-1).clip(max=V - 1).astype(np.int32)
    u = synth.philox_uniforms(7, 1, B, k + 1)[0]
    out = oracle.verify_level(lp, lq, tok, u, T, threads=4)
    expect = np.array([H.expected_accept_len_bottom(P[b], Q[b], k) for b in range(B)])
    diff = out["accepted_len"] - expect
    se = diff.std(ddof=1) / np.sqrt(B)
    assert abs(diff.mean()) < 3 * se, (diff.mean(), se)
    assert 0.5 < out["accepted_len"].mean() < k - 0.5          # the test is not vacuous


def test_constant_alpha_gives_the_capped_geometric_mean(oracle):
    """Every position shares one (P, Q) pair, so alpha is constant and the emitted length a + 1 has
    mean (1 - alpha^(m+1)) / (1 - alpha): the E[N] printed in the proof of Theorem 3.3 with n = m + 1
    trials and continuation probability alpha (its 1 - p)."""
    B, k, V = 6000, 5, 12
    r = _rng(8)
    zp = r.normal(0, 1.5, V).astype(np.float32)
    zq = (zp + r.normal(0, 1.0, V)).astype(np.float32)
    P, Q = H.prob_tables([zp[None], zq[None]], 1.0)
    alpha = np.minimum(P[0], Q[0]).sum()
    lp = np.broadcast_to(zp, (B, k + 1, V)).copy()
    lq = np.broadcast_to(zq, (B, k, V)).copy()
    tok = r.choice(V, size=(B, k), p=Q[0]).astype(np.int32)
    u = synth.philox_uniforms(8, 1, B, k + 1)[0]
    out = oracle.verify_level(lp, lq, tok, u, 1.0, threads=4)
    n = k + 1
    p = 1.0 - alpha
    paper_EN = (1.0 - (1.0 - p) ** n) / p
    emitted = out["accepted_len"] + 1
    se = emitted.std(ddof=1) / np.sqrt(B)
    assert abs(emitted.mean() - paper_EN) < 3 * se
    # and the variance of min(Geom, n): [a - (2n-1) a^n (1-a) - a^(2n)] / (1-a)^2, a = alpha
    a = alpha
    var = (a - (2 * n - 1) * a ** n * (1 - a) - a ** (2 * n)) / (1 - a) ** 2
    assert abs(emitted.var(ddof=1) - var) < 0.1 * var + 0.05


def test_chain_statistics_match_closed_forms(oracle):
    n, k, V, T, B = 3, (4, 5), 32, 1.0, 3000
    spec = synth.ChainSpec("t", n, B, V, torch.float32, k, T, 3.0, (0.6, 1.2), False)
    data = synth.make_chain(spec, seed=11)
    out = oracle.verify_chain(data["models"], data["k"], data["draft_tokens"], data["uniforms"], T, threads=4)
    tabs = [sp_softmax(m.double().numpy() / T, axis=-1) for m in data["models"]]
    e_bot = np.array([H.expected_accept_len_bottom(tabs[1][b], tabs[2][b], k[1]) for b in range(B)])
    e_top = np.array([H.expected_accept_len_second(tabs[0][b], tabs[1][b], tabs[2][b], k[0], k[1]) for b in range(B)])
    for l, e in ((1, e_bot), (0, e_top)):
        d = out["accepted_len"][l] - e
        se = d.std(ddof=1) / np.sqrt(B)
        assert abs(d.mean()) < 3 * se, (l, d.mean(), se)
    # hand-off bookkeeping: the block presented one level up is the stream below, capped
    assert (out["block_len"][0] == np.minimum(k[0], out["out_len"][1])).all()
    assert (out["block_len"][1] == k[1]).all()
    assert (out["out_len"] == out["accepted_len"] + 1).all()


def test_fused_variant_is_the_matmul_followed_by_the_level_rule(oracle):
    spec = synth.FusedSpec(B=3, k=2, V=40, d_p=16, d_q=8)
    d = synth.make_fused(spec, seed=5)
    out = oracle.verify_from_hidden(d["hidden_p"], d["W_p"], d["hidden_q"], d["W_q"], d["draft_tokens"],
                                    d["uniforms"], d["temperature"])
    # the contraction, element by element, from the stored bf16 values
    hp, wp = d["hidden_p"].double().numpy(), d["W_p"].double().numpy()
    ref = np.zeros((3, 3, 40))
    for b in range(3):
        for j in range(3):
            for v in range(40):
                ref[b, j, v] = sum(hp[b, j, i] * wp[v, i] for i in range(16))
    np.testing.assert_allclose(out["logits_p"].numpy(), ref, rtol=1e-12, atol=1e-12)
    again = oracle.verify_level(out["logits_p"], out["logits_q"][:, :2], d["draft_tokens"], d["uniforms"], 1.0)
    assert (again["accepted_len"] == out["accepted_len"]).all() and (again["next_token"] == out["next_token"]).all()


# ---------------------------------------------------------------- tie accounting of the GPU comparisons (host logic)
def test_sampling_tie_rule_with_tokens_lighter_than_the_band(oracle):
    """A sampling uniform within 1e-6 of a CDF edge is a counted tie.  Where the tokens next to that edge carry less
    mass than the band itself, several edges fall inside the band and the other side may land a few tokens away: still
    a tie if that token's own interval lies within the band of the uniform; never one if it lies further, or if the
    uniform is not near an edge of the oracle's token at all."""
    V, T = 64, 1.0
    z = np.full((1, 2, V), -60.0)
    z[0, :, 20] = 0.0                      # nearly all of the mass
    z[0, :, 40] = -0.5
    z[0, 0, 2:6] = -21.0                   # four tokens of ~5e-10 each at the start of the CDF, where float32 resolves them
    lq = np.full((1, 1, V), -60.0)
    lq[0, 0, 63] = 0.0                     # the drafter puts its mass on token 63: the draft is rejected
    P = H.prob_tables([z[0]], T)[0]
    Q = H.prob_tables([lq[0]], T)[0]
    w = np.maximum(P[0] - Q[0], 0.0)
    cdf = np.cumsum(w) / w.sum()
    u = np.float32(cdf[3] * (1 + 1e-3))    # just past the edge between tokens 3 and 4
    U = np.array([[0.999, u]], np.float32)
    out = oracle.verify_level(z, lq, np.array([[63]], np.int32), U, T)
    assert out["accepted_len"][0] == 0
    tok = int(out["next_token"][0])
    assert tok == 4 and out["sample_info"][0, 0] < 1e-6
    dist = lambda t: H.cdf_distance(w, float(u), t)
    margin, info = out["accept_margin"][0], out["sample_info"][0]
    assert H.compare_level(0, 3, 0, tok, margin, info) == "tie_sample"                     # the neighbour
    assert H.compare_level(0, 2, 0, tok, margin, info) == "mismatch"                       # adjacency alone: two tokens away
    assert H.compare_level(0, 2, 0, tok, margin, info, distance=dist) == "tie_sample"      # ... yet within 1e-6 in CDF units
    assert H.compare_level(0, 20, 0, tok, margin, info, distance=dist) == "tie_sample"     # the heavy token starts 5e-10 away
    assert H.compare_level(0, 40, 0, tok, margin, info, distance=dist) == "mismatch"       # far in CDF units
    assert H.compare_level(0, 1, 0, tok, margin, info, distance=dist) == "mismatch"        # a zero-mass token
    # a uniform in the middle of a heavy token's interval is no tie, whatever the other side returns
    U2 = np.array([[0.999, 0.3]], np.float32)
    out2 = oracle.verify_level(z, lq, np.array([[63]], np.int32), U2, T)
    assert out2["next_token"][0] == 20
    d2 = lambda t: H.cdf_distance(w, 0.3, t)
    assert H.compare_level(0, 5, 0, 20, out2["accept_margin"][0], out2["sample_info"][0], distance=d2) == "mismatch"
