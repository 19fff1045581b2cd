"""Input generators (Philox known answers, shapes, determinism) and the paper's printed closed form."""
import os

import numpy as np
import pytest
import torch

from paper_2510_26527_b200 import synth
from tests import helpers as H

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_philox_known_answers():
    for row in _rows("philox4x32_10_kat.txt"):
        w = [int(x, 16) for x in row]
        got = synth.philox4x32_10(np.array(w[0:4], dtype=np.uint32), (w[4], w[5]))
        assert [int(x) for x in got] == w[6:10]


def test_uniforms_are_open_interval_float32_and_counter_based():
    u = synth.philox_uniforms(0, 3, 5, 11)
    assert u.dtype == np.float32 and u.shape == (3, 5, 11)
    assert (u > 0).all() and (u < 1).all()
    # entry (l, b, j) depends only on its own counter: a larger grid and an offset batch agree with it
    u2 = synth.philox_uniforms(0, 4, 9, 12)
    assert (u2[:3, :5, :11] == u).all()
    u3 = synth.philox_uniforms(0, 3, 2, 11, batch_offset=3)
    assert (u3 == u[:, 3:5]).all()
    assert (synth.philox_uniforms(1, 3, 5, 11) != u).any()
    big = synth.philox_uniforms(2, 1, 1, 200000).ravel()
    assert abs(big.mean() - 0.5) < 3 / np.sqrt(12 * big.size) and abs(big.var() - 1 / 12) < 1e-3


def test_config_shapes_and_byte_counts():
    c1, c2, c3, c5 = (synth.config(n) for n in ("cfg1", "cfg2", "cfg3", "cfg5"))
    assert c1.rows == (5, 4) and c1.logits_bytes() == 1_152_000
    assert c2.rows == (10, 9, 8) and c2.logits_bytes() == 1_728_000
    assert c3.rows == (7, 7, 6) and c3.logits_bytes() == 64 * 20 * 128256 * 2
    assert c5.rows == (5, 7, 11, 10) and c5.logits_bytes() == 256 * 33 * 152064 * 2
    f = synth.FusedSpec()
    assert f.weight_bytes() == 2 * 32000 * 6144 and f.flops() == 2 * 288 * 32000 * 6144


def test_make_chain_is_seeded_and_shaped():
    spec = synth.scaled(synth.config("cfg3"), B=2, V=512)
    a, b = synth.make_chain(spec, 3), synth.make_chain(spec, 3)
    c = synth.make_chain(spec, 4)
    assert [tuple(m.shape) for m in a["models"]] == [(2, 7, 512), (2, 7, 512), (2, 6, 512)]
    assert all(m.dtype == torch.bfloat16 for m in a["models"])
    assert all(torch.equal(x, y) for x, y in zip(a["models"], b["models"]))
    assert torch.equal(a["draft_tokens"], b["draft_tokens"]) and torch.equal(a["uniforms"], b["uniforms"])
    assert not torch.equal(a["models"][0], c["models"][0])
    assert a["draft_tokens"].shape == (2, 6) and a["draft_tokens"].dtype == torch.int32
    assert a["uniforms"].shape == (2, 2, 7) and a["uniforms"].dtype == torch.float32
    # peaked rows: about 1 % of the entries of the target sit ~8 above the N(0, 4^2) bulk
    m1 = a["models"][0].float()
    assert (m1 > 12).float().mean() > 0.002          # 0.00135 without the boost, ~0.0029 with it
    # cumulative noise in cfg5: M3 - M2 has the same spread as M2 - M1
    s5 = synth.scaled(synth.config("cfg5", sigma=0.5), B=2, V=4096)
    d5 = synth.make_chain(s5, 1)
    m = [x.float() for x in d5["models"]]
    assert abs((m[1][:, :5] - m[0]).std() - 0.5) < 0.05 and abs((m[2][:, :7] - m[1]).std() - 0.5) < 0.05
    assert abs((m[2][:, :5] - m[0]).std() - 0.5 * np.sqrt(2)) < 0.05


def test_make_fused_tracks_the_target():
    spec = synth.FusedSpec(B=2, k=3, V=2048, d_p=256, d_q=128)
    d = synth.make_fused(spec, 0)
    lp = d["hidden_p"].float() @ d["W_p"].float().t()
    lq = d["hidden_q"].float() @ d["W_q"].float().t()
    assert abs(lp.std() - 3.0) < 0.3 and abs(lq.std() - 3.0) < 0.3
    assert torch.corrcoef(torch.stack([lp.flatten(), lq.flatten()]))[0, 1] > 0.9
    assert d["draft_tokens"].shape == (2, 3) and d["uniforms"].shape == (2, 4)


@pytest.mark.parametrize("row", _rows("theorem33_expected_length.txt"))
def test_expected_emitted_length_printed_in_theorem_3_3(oracle, row):
    """Exact enumeration of the oracle on a two-token vocabulary with constant acceptance probability
    alpha = 1 - p reproduces E[N] = (1 - (1 - p)^n) / p for n = block length + 1."""
    p, n, EN = float(row[0]), int(row[1]), float(row[2])
    k = n - 1
    if k == 0:
        assert abs(EN - 1.0) < 1e-14
        return
    alpha = 1.0 - p
    lp = np.tile(np.array([0.0, -np.inf]), (k + 1, 1))                    # P = (1, 0)
    lq = np.tile(np.log(np.array([alpha, 1.0 - alpha])), (k, 1))           # Q = (alpha, 1 - alpha): sum min = alpha
    P, Q = H.prob_tables([lp, lq], 1.0)
    mean_emitted = 0.0
    for weight, U, draft, trace in H.enumerate_chain([P, Q], [k], 2):
        out = oracle.verify_level(lp[None], lq[None], np.array([draft], np.int32), U.astype(np.float32), 1.0)
        (_, _, a, stream), = trace
        assert out["accepted_len"][0] == a and out["next_token"][0] == stream[-1]
        mean_emitted += weight * (out["accepted_len"][0] + 1)
    assert abs(mean_emitted - EN) < 1e-9
