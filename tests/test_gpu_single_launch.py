"""The single-launch path of the chain (row stream with every sequence's decisions trailing it) on shapes that the
automatic choice would send through two launches, and against those two launches.

polyspec_verify_chain / polyspec_verify_level take the single launch for rows of 8 KiB and more, so the full-size
configurations in test_gpu_parity.py already run it.  Here it is forced (polyspec_*_single_launch) on small,
ragged and degenerate shapes, every result compared with the CPU oracle, and on several shapes with the two
halves polyspec_chain_row_stats + polyspec_chain_walk, which must agree bit for bit: both paths use the same
partials, the same merge, the same residual arithmetic and the same scan order, only the schedule differs.
"""
import numpy as np
import pytest
import torch

from paper_2510_26527_b200 import binding, buildlib, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
KEYS = ("accepted_len", "block_len", "out_tokens", "out_len")


@pytest.fixture(scope="module", autouse=True)
def _lib():
    buildlib.build()
    binding.load_library()
    assert torch.cuda.is_available()


def _np(out):
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def _single(d):
    return _np(binding.polyspec_verify_chain(d["models"], d["k"], d["draft_tokens"], d["uniforms"], d["temperature"], single_launch=True))


def _halves(d):
    call = binding.ChainCall(d["models"], d["k"], d["draft_tokens"], d["uniforms"], d["temperature"])
    call.row_stats()
    return _np(call.walk())


def _oracle(oracle, d):
    return oracle.verify_chain([m.cpu() for m in d["models"]], d["k"], d["draft_tokens"].cpu(), d["uniforms"].cpu(), d["temperature"], threads=8)


def _check(counts, bad, n, what):
    print(f"[parity] single launch, {what}: {counts}")
    assert not bad, (what, bad[:5])
    assert counts["tie_accept"] + counts["tie_sample"] <= max(2, n // 2000), counts


@pytest.mark.parametrize("name,B,V,sigma", [("cfg2", 24, 4096, None), ("cfg3", 16, 10000, None), ("cfg5", 12, 8200, 0.5),
                                            ("cfg5", 12, 24, 2.0), ("cfg3", 300, 6152, None), ("cfg5", 40, 20000, 0.25),
                                            ("cfg1", 3, 32000, None), ("cfg2", 1, 32000, None)])
def test_forced_single_launch_against_the_oracle_and_the_two_launches(oracle, name, B, V, sigma):
    spec = synth.scaled(synth.config(name, sigma=sigma), B=B, V=V)
    d = synth.make_chain(spec, seed=31, device=DEV)
    one = _single(d)
    assert one["device_status"][0] == 0
    counts, bad = H.compare_chain(one, _oracle(oracle, d))
    _check(counts, bad, B * sum(spec.k), f"{name} B={B} V={V}")
    two = _halves(d)
    for key in KEYS:
        assert (one[key] == two[key]).all(), key


def test_forced_single_launch_random_shapes(oracle):
    rng = np.random.default_rng(20251027)
    total = {"exact": 0, "tie_accept": 0, "tie_sample": 0, "mismatch": 0}
    for case in range(40):
        n_models = int(rng.integers(2, 6))
        B = int(rng.integers(1, 70))
        V = 8 * int(rng.integers(1, 3000))
        k = tuple(int(x) for x in rng.integers(1, 13, size=n_models - 1))
        if case % 8 == 0:
            k = k[:-1] + (32,)
        dtype = torch.float32 if rng.random() < 0.5 else torch.bfloat16
        T = float(rng.choice([0.5, 0.8, 1.0, 1.7]))
        sig = tuple(float(x) for x in rng.uniform(0.3, 2.5, size=n_models - 1))
        spec = synth.ChainSpec(f"rand{case}", n_models, B, V, dtype, k, T, 2.5, sig, bool(rng.random() < 0.5))
        d = synth.make_chain(spec, seed=2000 + case, device=DEV)
        one = _single(d)
        counts, bad = H.compare_chain(one, _oracle(oracle, d))
        assert not bad, (case, n_models, B, V, k, dtype, T, bad[:3])
        for key in total:
            total[key] += counts[key]
        if case % 4 == 0:
            two = _halves(d)
            for key in KEYS:
                assert (one[key] == two[key]).all(), (case, key)
        if n_models == 2:                                        # the single-level call: ragged block lengths, probabilities
            bl = torch.from_numpy(rng.integers(0, k[0] + 1, size=B).astype(np.int32)).to(DEV)
            lq = d["models"][1][:, : k[0]].contiguous()
            u = d["uniforms"][0].contiguous()
            lv = _np(binding.polyspec_verify_level(d["models"][0], lq, d["draft_tokens"], u, T, block_len=bl, want_probs=True, single_launch=True))
            ol = oracle.verify_level(d["models"][0].cpu(), d["models"][1].cpu(), d["draft_tokens"].cpu(), u.cpu(), T, block_len=bl.cpu())
            c2, bad2 = H.compare_level_batch(lv["accepted_len"], lv["next_token"], ol)
            assert not bad2, (case, B, V, k, bad2[:3])
            # the two-launch path reports the same probabilities, also past the first rejection and 0 past block_len
            tw = _two_launch_level(d["models"][0], lq, d["draft_tokens"], u, T, bl)
            assert np.array_equal(lv["p_at_draft"], tw["p_at_draft"]) and np.array_equal(lv["q_at_draft"], tw["q_at_draft"]), case
            assert np.array_equal(lv["accepted_len"], tw["accepted_len"]) and np.array_equal(lv["next_token"], tw["next_token"])
    print(f"[parity] single launch, random shapes: {total}")
    assert total["tie_accept"] + total["tie_sample"] <= 4


def _two_launch_level(lp, lq, tok, u, T, bl):
    """The level through the two halves of the chain call (a two-model chain), plus the probabilities of the walk."""
    B, k = tok.shape
    if lp.shape[2] * lp.element_size() < 8192:                  # short rows: the automatic choice is the two launches
        return _np(binding.polyspec_verify_level(lp, lq, tok, u, T, block_len=bl, want_probs=True))
    # long rows: the automatic choice would be the single launch again, so go through the static-scratch entry point,
    # which always takes the two launches
    out = {"accepted_len": torch.empty(B, dtype=torch.int32, device=DEV), "next_token": torch.empty(B, dtype=torch.int32, device=DEV),
           "p_at_draft": torch.empty((B, k), device=DEV), "q_at_draft": torch.empty((B, k), device=DEV)}
    binding.polyspec_verify_level_static(lp, lq, tok, u, T, out, block_len=bl)
    return _np(out)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V,k", [(8, 1), (1000, 2), (4104, 5), (16384 + 8, 3)])
def test_forced_single_launch_level_every_branch(oracle, dtype, V, k):
    B = 512
    spec = synth.ChainSpec("tiny", 2, B, V, dtype, (k,), 0.9, 2.0, (1.2,), False)
    d = synth.make_chain(spec, seed=V + k, device=DEV)
    lp, lq = d["models"]
    out = _np(binding.polyspec_verify_level(lp, lq, d["draft_tokens"], d["uniforms"][0], 0.9, want_probs=True, single_launch=True))
    ora = oracle.verify_level(lp.cpu(), lq.cpu(), d["draft_tokens"].cpu(), d["uniforms"][0].cpu(), 0.9, threads=8)
    counts, bad = H.compare_level_batch(out["accepted_len"], out["next_token"], ora)
    _check(counts, bad, B * (k + 1), f"level V={V} k={k} {dtype}")
    assert out["device_status"][0] == 0
    assert set(np.unique(ora["accepted_len"])) == set(range(k + 1))
    tol = 1e-5 if dtype == torch.float32 else 2e-3
    m = np.isfinite(ora["p_at"])
    np.testing.assert_allclose(out["p_at_draft"][m], ora["p_at"][m], rtol=tol, atol=1e-30)
    np.testing.assert_allclose(out["q_at_draft"][m], ora["q_at"][m], rtol=tol, atol=1e-30)


def test_forced_single_launch_unusable_inputs_and_vanishing_residual(oracle):
    B, k, V = 8, 3, 1024
    g = torch.Generator(device=DEV).manual_seed(3)
    lp = torch.randn((B, k + 1, V), generator=g, device=DEV)
    lq = lp[:, :k].clone() + 0.5 * torch.randn((B, k, V), generator=g, device=DEV)
    tok = torch.randint(0, V, (B, k), generator=g, device=DEV, dtype=torch.int32)
    u = torch.full((B, k + 1), 1e-6, device=DEV)
    tok[1, 0] = V
    tok[2, 2] = -1
    lp[3, 1, 17] = float("nan")
    lq[4, 0] = float("-inf")
    lp[5, k, 5] = float("inf")
    out = _np(binding.polyspec_verify_level(lp, lq, tok, u, 1.0, single_launch=True))
    ora = oracle.verify_level(lp.cpu(), lq.cpu(), tok.cpu(), u.cpu(), 1.0)
    assert out["device_status"][0] == binding.ERR_BAD_INPUT_ON_DEVICE
    for b in range(B):
        if ora["status"][b] != 0:
            assert out["accepted_len"][b] == -1 and out["next_token"][b] == -1, b
        else:
            assert out["accepted_len"][b] == ora["accepted_len"][b] and out["next_token"][b] == ora["next_token"][b], b
    # a chain in which an upper level meets the bad row: that level and the ones above report -1, the ones below do not
    spec = synth.scaled(synth.config("cfg5", sigma=0.25), B=6, V=9000)
    d = synth.make_chain(spec, seed=8, device=DEV)
    d["models"][1][2, 0, 100] = float("nan")                     # M_2's first row of sequence 2
    one = _single(d)
    ora = _oracle(oracle, d)
    two = _halves(d)
    assert one["device_status"][0] == binding.ERR_BAD_INPUT_ON_DEVICE
    for key in KEYS:
        assert (one[key] == two[key]).all(), key
        assert (one[key][:, 2] == ora[key][:, 2]).all(), key
    assert one["accepted_len"][2, 2] >= 0 and one["accepted_len"][1, 2] == -1 and one["accepted_len"][0, 2] == -1
    # p == q at the rejected row, the rejection forced by an accept uniform above 1: the residual is 0 everywhere and P
    # is sampled instead; long rows (the pass goes through the job queue twice) and short ones (summed on the spot)
    for Vv in (16384 + 512, 2048):
        lp2 = torch.randn((6, 3, Vv), generator=g, device=DEV) * 2
        lq2 = lp2[:, :2].clone()
        tok2 = torch.randint(0, Vv, (6, 2), generator=g, device=DEV, dtype=torch.int32)
        u2 = torch.from_numpy(synth.philox_uniforms(4, 1, 6, 3)[0]).to(DEV)
        u2[:, 0] = 1.5
        o2 = _np(binding.polyspec_verify_level(lp2, lq2, tok2, u2, 1.0, single_launch=True))
        r2 = oracle.verify_level(lp2.cpu(), lq2.cpu(), tok2.cpu(), u2.cpu(), 1.0)
        assert (r2["fallback"] == 1).all() and (o2["accepted_len"] == 0).all()
        assert (o2["next_token"] == r2["next_token"]).all(), (Vv, o2["next_token"], r2["next_token"])


def test_config3_and_config5_single_launch_equals_two_launches():
    for spec, seed in ((synth.config("cfg3"), 0), (synth.config("cfg5", sigma=1.0), 1), (synth.config("cfg5", sigma=0.25), 2)):
        d = synth.make_chain(spec, seed=seed, device=DEV)
        one = _single(d)
        two = _halves(d)
        assert one["device_status"][0] == 0
        for key in KEYS:
            assert (one[key] == two[key]).all(), (spec.name, key)


def test_outputs_do_not_depend_on_the_schedule():
    """Which warp runs which state machine, and in which order residual jobs are served, changes from launch to launch;
    the outputs may not."""
    spec = synth.scaled(synth.config("cfg5", sigma=0.5), B=96, V=40000)
    d = synth.make_chain(spec, seed=5, device=DEV)
    first = _single(d)
    for _ in range(5):
        again = _single(d)
        for key in KEYS:
            assert (first[key] == again[key]).all(), key


def test_copy_wait_that_runs_out_reports_timeout_and_leaves_the_device_usable(oracle):
    """The give-up path of the row-statistics kernel, in the safe form: the wait for a copy is given a single poll, which a
    copy from HBM cannot meet; the warps record POLYSPEC_ERR_TIMEOUT, still wait (full limit) for the copies they
    have in flight, and return.  The next ordinary call on the same device and workspace is exact."""
    spec = synth.scaled(synth.config("cfg3"), B=8, V=65536)
    d = synth.make_chain(spec, seed=17, device=DEV)
    call = binding.ChainCall(d["models"], d["k"], d["draft_tokens"], d["uniforms"], d["temperature"])
    call.row_stats_wait_limit(1)
    torch.cuda.synchronize()
    assert int(call.device_status.item()) == binding.ERR_TIMEOUT
    call.device_status.zero_()
    call.row_stats()
    out = _np(call.walk())
    assert out["device_status"][0] == 0
    counts, bad = H.compare_chain(out, _oracle(oracle, d))
    assert not bad and counts["exact"] == 8 * 2
    with pytest.raises(binding.PolyspecError):
        call.row_stats_wait_limit(0)
