"""Test-side helpers: library softmax tables, exact branch enumeration, closed forms, tie accounting.

Nothing here is used by the product.  The enumeration drives the oracle through every
branch of the verification rule with exact weights ("branch-midpoint quadrature"): each
accept uniform is put at the midpoint of its accept region (0, t] or reject region (t, 1)
and weighted by that region's length, the sampling uniform at the midpoint of each token's
CDF interval and weighted by the interval's length.
"""
from __future__ import annotations

import itertools

import numpy as np
from scipy.special import softmax as sp_softmax


def prob_tables(models, T):
    """float64 softmax tables [rows_i, V] per model from (float64-convertible) logits [rows_i, V]."""
    return [sp_softmax(np.asarray(m, dtype=np.float64) / T, axis=-1) for m in models]


def level_branches(P, Q, stream, k_l):
    """All (a, token, weight, accept_uniforms, sampling_uniform) of one level given the incoming stream."""
    m = min(k_l, len(stream))
    out = []
    for a in range(m + 1):
        w = 1.0
        ua = [0.5] * k_l
        ok = True
        for j in range(a):
            t = min(1.0, P[j, stream[j]] / Q[j, stream[j]])
            w *= t
            ua[j] = t / 2.0
        if a < m:
            t = min(1.0, P[a, stream[a]] / Q[a, stream[a]])
            if t >= 1.0:
                ok = False
            else:
                w *= 1.0 - t
                ua[a] = (t + 1.0) / 2.0
            D = np.maximum(P[a] - Q[a], 0.0)
        else:
            D = P[m].copy()
        if not ok or w == 0.0:
            continue
        D = D / D.sum()
        cdf = np.concatenate([[0.0], np.cumsum(D)])
        for v in range(len(D)):
            if D[v] <= 0.0:
                continue
            out.append((a, v, w * D[v], list(ua), 0.5 * (cdf[v] + cdf[v + 1])))
    return m, out


def enumerate_chain(tables, k, V):
    """Yield (weight, uniforms [L, kmax+1], draft tokens, expected per-level (m, a, stream)) over all branches."""
    n = len(tables)
    L = n - 1
    kmax = max(k)

    def rec(l, stream, weight, U, trace):
        if l < 0:
            yield weight, U, trace
            return
        m, branches = level_branches(tables[l], tables[l + 1], stream, k[l])
        for a, v, w, ua, us in branches:
            U2 = U.copy()
            U2[l, :k[l]] = ua
            U2[l, kmax] = us
            yield from rec(l - 1, stream[:a] + [v], weight * w, U2, trace + [(l, m, a, stream[:a] + [v])])

    Qb = tables[n - 1]
    for draft in itertools.product(range(V), repeat=k[L - 1]):
        w = 1.0
        for j, x in enumerate(draft):
            w *= Qb[j, x]
        U = np.full((L, kmax + 1), 0.5)
        for weight, U2, trace in rec(L - 1, list(draft), w, U, []):
            yield weight, U2, list(draft), trace


def expected_accept_len_bottom(P, Q, m):
    """E[a] = sum_j prod_{i<=j} alpha_i with alpha_i = sum_v min(P_i, Q_i): the bottom level's closed form.

    With a constant alpha this is alpha (1 - alpha^m) / (1 - alpha); counting the replacement/bonus
    token as well gives (1 - alpha^(m+1)) / (1 - alpha), the capped-geometric mean in the proof of
    Theorem 3.3 with n = m + 1 and continuation probability alpha.
    """
    alpha = np.minimum(P[:m], Q[:m]).sum(axis=-1)
    return float(np.cumprod(alpha).sum())


def expected_accept_len_second(P1, P2, Q3, k1, k2):
    """E[a] of the level above the bottom one (three consecutive models M_1, M_2, M_3 = drafter).

    Position i < j must carry a draft token accepted by both levels, probability
    gamma_i = sum_v min(Q3_i, P2_i)(v) min(1, P1_i(v) / P2_i(v)); the token at position j then has
    law P2_j, so it passes with alpha_j = sum_v min(P1_j, P2_j).  j runs to min(k1, k2 + 1).
    """
    J = min(k1, k2 + 1)
    total, surv = 0.0, 1.0
    for j in range(J):
        alpha = np.minimum(P1[j], P2[j]).sum()
        total += surv * alpha
        if j < k2:
            ratio = np.minimum(1.0, P1[j] / P2[j])
            surv *= (np.minimum(Q3[j], P2[j]) * ratio).sum()
    return float(total)


TIE_BAND = 1e-6


def compare_level(gpu_a, gpu_next, ora_a, ora_next, accept_margin, sample_info, band=TIE_BAND, distance=None):
    """Classify one (level, sequence) result against the oracle.

    Returns "exact", "tie_accept" (accept decisions differ at a position whose uniform lies within
    `band` of min(1, P/Q)), "tie_sample" (same accepted length, the sampling uniform lies within
    `band`, in normalised CDF units, of an edge of the oracle's token's interval, and the GPU token
    is the neighbouring positive-mass token -- or, where tokens carry less mass than the band itself
    so that several edges fall inside it, a token whose own interval lies within `band` of the
    uniform: `distance(token)` gives that distance under the oracle's float64 weights) or "mismatch".
    """
    if gpu_a == ora_a and gpu_next == ora_next:
        return "exact"
    if gpu_a != ora_a:
        j = min(gpu_a, ora_a)
        if 0 <= j < len(accept_margin) and np.isfinite(accept_margin[j]) and accept_margin[j] <= band:
            return "tie_accept"
        return "mismatch"
    margin, _, prev, succ = sample_info
    if margin <= band and gpu_next >= 0:
        if gpu_next in (int(prev), int(succ)):
            return "tie_sample"
        if distance is not None and distance(gpu_next) <= band:
            return "tie_sample"
    return "mismatch"


def chain_sample_distance(oracle, models, uniforms, temperature, ora, seq_map=None):
    """distance(l, b)(token) for compare_chain: how far, in normalised CDF units, the sampling uniform of level l,
    sequence b lies from `token`'s inverse-CDF interval under the oracle's float64 weights (the residual of the row
    pair at the oracle's accepted length, or the bonus row).  models: CPU tensors [B, rows, V]; seq_map maps the
    index b of `ora` to the row of `models` / `uniforms` (identity if None)."""
    kmax = uniforms.shape[-1] - 1

    def at(l, b):
        def distance(token):
            bb = b if seq_map is None else seq_map[b]
            a, m = int(ora["accepted_len"][l, b]), int(ora["block_len"][l, b])
            P = oracle.softmax_row(models[l][bb, a], temperature)
            w = np.maximum(P - oracle.softmax_row(models[l + 1][bb, a], temperature), 0.0) if a < m else P
            if not (w.sum() > 0.0):
                w = P
            return cdf_distance(w, float(uniforms[l, bb, kmax]), int(token))
        return distance
    return at


def compare_chain(gpu, ora, seqs=None, band=TIE_BAND, distance=None):
    """Compare chain outputs (dicts of numpy arrays [L, B, ...]) sequence by sequence, bottom level first.

    After a counted tie the two sides walk different streams, so the levels above it are skipped
    (counted as "skipped_after_tie").  `distance(l, b)` returns compare_level's distance function
    (see chain_sample_distance).  Returns a dict of counts and a list of mismatch descriptions.
    """
    L, B = ora["accepted_len"].shape
    counts = {"exact": 0, "tie_accept": 0, "tie_sample": 0, "mismatch": 0, "skipped_after_tie": 0}
    bad = []
    for b in (range(B) if seqs is None else seqs):
        for l in range(L - 1, -1, -1):
            kind = compare_level(int(gpu["accepted_len"][l, b]), int(gpu["out_tokens"][l, b, max(int(gpu["accepted_len"][l, b]), 0)]),
                                 int(ora["accepted_len"][l, b]), int(ora["out_tokens"][l, b, max(int(ora["accepted_len"][l, b]), 0)]),
                                 ora["accept_margin"][l, b], ora["sample_info"][l, b], band,
                                 None if distance is None else distance(l, b))
            if kind == "exact":
                same = (gpu["block_len"][l, b] == ora["block_len"][l, b] and gpu["out_len"][l, b] == ora["out_len"][l, b]
                        and (gpu["out_tokens"][l, b] == ora["out_tokens"][l, b]).all())
                if not same:
                    kind = "mismatch"
            counts[kind] += 1
            if kind == "mismatch":
                bad.append((b, l, int(gpu["accepted_len"][l, b]), int(ora["accepted_len"][l, b]),
                            gpu["out_tokens"][l, b].tolist(), ora["out_tokens"][l, b].tolist()))
                break
            if kind != "exact":
                counts["skipped_after_tie"] += l
                break
    return counts, bad


def compare_level_batch(gpu_a, gpu_next, ora, seqs=None, band=TIE_BAND):
    counts = {"exact": 0, "tie_accept": 0, "tie_sample": 0, "mismatch": 0}
    bad = []
    B = len(ora["accepted_len"])
    for b in (range(B) if seqs is None else seqs):
        kind = compare_level(int(gpu_a[b]), int(gpu_next[b]), int(ora["accepted_len"][b]), int(ora["next_token"][b]),
                             ora["accept_margin"][b], ora["sample_info"][b], band)
        counts[kind] += 1
        if kind == "mismatch":
            bad.append((b, int(gpu_a[b]), int(gpu_next[b]), int(ora["accepted_len"][b]), int(ora["next_token"][b])))
    return counts, bad


def cdf_distance(weights, u, token):
    """Distance, in normalised CDF units, from the uniform u to the inverse-CDF interval of `token`
    under the (unnormalised, float64) weights; 0 if u falls inside it.  inf for a zero-mass token."""
    w = np.asarray(weights, dtype=np.float64)
    if token < 0 or token >= len(w) or not (w[token] > 0.0):
        return float("inf")
    c = np.cumsum(w)
    total = c[-1]
    lo = (c[token] - w[token]) / total
    hi = c[token] / total
    return float(max(lo - u, u - hi, 0.0))
