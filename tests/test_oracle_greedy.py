"""Pins of the oracle's greedy-matching rule (Section 3.1 names greedy matching as a verification rule,
Section 4.5 compares it with speculative sampling).

Greedy matching has a plain definition, so the pins are that definition through library routines and a
cross-check against the independent sampling oracle in the limit where the two rules coincide:
  - the emitted stream equals the row-wise numpy arg max of the verifier's rows, for its length;
  - the accepted length is the number of leading block tokens that equal those arg maxes;
  - with arg-max drafts and a temperature so low that every softmax is one-hot, the *sampling* oracle
    (different C routine, different arithmetic) emits the same lengths and tokens for any uniforms.
"""
import numpy as np
import pytest
import torch

from paper_2510_26527_b200 import synth


def _rng(seed):
    return np.random.default_rng(seed)


def _drafts_with_matching_prefixes(top, r, V):
    """Block tokens equal to the verifier's arg max for a random prefix length, then a different token."""
    B, k1 = top.shape
    k = k1 - 1
    tok = top[:, :k].copy()
    pref = r.integers(0, k + 1, size=B)
    for b in range(B):
        for j in range(pref[b], k):
            if j == pref[b] or r.random() < 0.5:
                tok[b, j] = (top[b, j] + 1 + r.integers(0, V - 1)) % V          # never the arg max
    return tok.astype(np.int32), pref


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f64"])
def test_single_level_is_the_rowwise_argmax(oracle, dtype):
    B, k, V = 200, 6, 97
    r = _rng(21)
    z = r.normal(0, 3, (B, k + 1, V))
    if dtype == "f32":
        lp = z.astype(np.float32)
    elif dtype == "f64":
        lp = z
    else:
        lp = torch.from_numpy(z).to(torch.bfloat16)
    vals = lp.double().numpy() if dtype == "bf16" else np.asarray(lp, dtype=np.float64)
    top = vals.argmax(-1)                                   # numpy: first index of the maximum
    tok, pref = _drafts_with_matching_prefixes(top, r, V)
    out = oracle.verify_chain_greedy([lp, None], [k], tok)
    assert (out["status"] == 0).all()
    assert (out["accepted_len"][0] == pref).all()
    assert set(pref.tolist()) == set(range(k + 1))          # every accepted length occurs
    for b in range(B):
        a = pref[b]
        assert (out["out_tokens"][0, b, :a + 1] == top[b, :a + 1]).all()      # the verifier's own greedy tokens
        assert (out["out_tokens"][0, b, a + 1:] == -1).all()
    assert (out["out_len"][0] == pref + 1).all() and (out["block_len"][0] == k).all()


def test_ties_go_to_the_lowest_index_and_bad_rows_are_reported(oracle):
    V, k = 16, 2
    lp = np.zeros((4, k + 1, V), dtype=np.float32)
    lp[0, 0, [3, 9]] = 5.0                                   # tie: index 3 wins
    lp[1, 0, 2] = np.nan
    lp[2, 1, 7] = np.inf
    lp[3, 0, :] = -np.inf
    tok = np.array([[3, 0], [0, 0], [0, 0], [0, 0]], dtype=np.int32)
    out = oracle.verify_chain_greedy([lp, None], [k], tok)
    assert out["status"].tolist() == [0, 1, 1, 2]
    assert out["accepted_len"][0, 0] == 2 and out["out_tokens"][0, 0].tolist() == [3, 0, 0]
    assert (out["accepted_len"][0, 1:] == -1).all()
    tok_bad = np.array([[V, 0]] * 4, dtype=np.int32)
    assert oracle.verify_chain_greedy([lp, None], [k], tok_bad)["status"][0] == 3


def test_chain_streams_are_each_verifiers_greedy_tokens(oracle):
    n, k, V, B = 4, (3, 4, 5), 64, 300
    spec = synth.ChainSpec("g", n, B, V, torch.float32, k, 1.0, 3.0, (0.3, 0.3, 0.3), True)
    d = synth.make_chain(spec, seed=22)
    draft = d["models"][3].double().numpy().argmax(-1).astype(np.int32)       # a greedy drafter
    out = oracle.verify_chain_greedy(d["models"], d["k"], draft)
    tops = [m.double().numpy().argmax(-1) for m in d["models"]]
    stream_len = np.full(B, k[2])
    stream = draft.copy()
    for l in (2, 1, 0):
        m = np.minimum(k[l], stream_len)
        assert (out["block_len"][l] == m).all()
        for b in range(B):
            a = 0
            while a < m[b] and stream[b, a] == tops[l][b, a]:
                a += 1
            assert out["accepted_len"][l, b] == a
            assert (out["out_tokens"][l, b, :a + 1] == tops[l][b, :a + 1]).all()
        new_len = out["out_len"][l]
        width = max(stream.shape[1], int(new_len.max()))
        nxt = np.full((B, width), -1, dtype=np.int64)
        for b in range(B):
            nxt[b, :new_len[b]] = out["out_tokens"][l, b, :new_len[b]]
        stream, stream_len = nxt, new_len
    assert len(set(out["accepted_len"][0].tolist())) >= 3                      # not vacuous


def test_sampling_rule_reduces_to_greedy_matching_at_low_temperature(oracle):
    """Arg-max drafts and T so low that every softmax is one-hot (logit gaps >= 1, T = 0.01): the
    sampling oracle's accept test becomes x == argmax p, its residual and bonus rows become one-hot at
    argmax p, whatever the uniforms.  Two independent routines must agree."""
    n, k, V, B = 3, (4, 4), 24, 400
    r = _rng(23)
    models = []
    base = np.round(r.normal(0, 2, (B, 5, V)))
    for i in range(n):
        z = base + np.round(r.normal(0, 0.8, (B, 5, V)))
        win = r.integers(0, V, size=(B, 5))
        np.put_along_axis(z, win[..., None], z.max(-1, keepdims=True) + 1.0, axis=-1)     # unique maximum, gap >= 1
        models.append(z[:, : (k[i] + 1 if i < n - 1 else k[-1])].astype(np.float32))
    draft = models[2].argmax(-1).astype(np.int32)
    u = synth.philox_uniforms(23, n - 1, B, max(k) + 1)
    samp = oracle.verify_chain(models, list(k), draft, u, 0.01, threads=4)
    greedy = oracle.verify_chain_greedy(models, list(k), draft, threads=4)
    for key in ("accepted_len", "block_len", "out_len", "out_tokens"):
        assert (samp[key] == greedy[key]).all(), key
    assert len(set(greedy["accepted_len"][1].tolist())) >= 3
