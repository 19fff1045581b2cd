"""GPU-vs-oracle parity of the logits path, through the C ABI, on the same seeded inputs.

Bar: accepted lengths, block lengths, stream lengths and every emitted token bit-exact, except where
a uniform lies within 1e-6 of its decision threshold (accept tests: |u - min(1, P/Q)|; sampling:
distance to the chosen token's CDF edge in normalised units, and the GPU token must then be the
neighbouring positive-mass token).  Such ties are counted, printed and bounded.  Softmax
probabilities at the drafted tokens agree to 1e-5 relative (fp32 logits) / 2e-3 (bf16 logits).
"""
import numpy as np
import pytest
import torch

from paper_2510_26527_b200 import binding, buildlib, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _lib():
    buildlib.build()
    binding.load_library()
    assert torch.cuda.is_available()


def _np(out):
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def _cpu(models):
    return [m.cpu() for m in models]


def _run_chain(data):
    return _np(binding.polyspec_verify_chain(data["models"], data["k"], data["draft_tokens"], data["uniforms"], data["temperature"]))


def _oracle_chain(oracle, data, seqs=None, threads=8):
    return oracle.verify_chain(_cpu(data["models"]), data["k"], data["draft_tokens"].cpu(), data["uniforms"].cpu(),
                               data["temperature"], threads=threads, seqs=seqs)


def _assert_parity(counts, bad, n_decisions, what):
    ties = counts["tie_accept"] + counts["tie_sample"]
    print(f"[parity] {what}: {counts}")
    assert not bad, f"{what}: mismatches outside the 1e-6 band: {bad[:5]}"
    assert ties <= max(2, n_decisions // 2000), f"{what}: implausibly many ties {counts}"


# ------------------------------------------------------------------ single level, tiny shapes, every branch
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V,k", [(8, 1), (64, 3), (1000, 2), (2048, 4), (4104, 5)])
def test_level_tiny_shapes_every_branch(oracle, dtype, V, k):
    B = 512
    spec = synth.ChainSpec("tiny", 2, B, V, dtype, (k,), 0.9, 2.0, (1.2,), False)
    d = synth.make_chain(spec, seed=V + k, device=DEV)
    lp, lq = d["models"]
    out = _np(binding.polyspec_verify_level(lp, lq, d["draft_tokens"], d["uniforms"][0], 0.9, want_probs=True))
    ora = oracle.verify_level(lp.cpu(), lq.cpu(), d["draft_tokens"].cpu(), d["uniforms"][0].cpu(), 0.9, threads=8)
    counts, bad = H.compare_level_batch(out["accepted_len"], out["next_token"], ora)
    _assert_parity(counts, bad, B * (k + 1), f"level V={V} k={k} {dtype}")
    assert out["device_status"][0] == 0
    assert set(np.unique(ora["accepted_len"])) == set(range(k + 1))        # every accepted length occurs
    # probabilities at the drafted tokens (the oracle fills positions up to the first rejection)
    tol = 1e-5 if dtype == torch.float32 else 2e-3
    m = np.isfinite(ora["p_at"])
    np.testing.assert_allclose(out["p_at_draft"][m], ora["p_at"][m], rtol=tol, atol=1e-30)
    np.testing.assert_allclose(out["q_at_draft"][m], ora["q_at"][m], rtol=tol, atol=1e-30)


def test_level_block_len_zero_to_k_and_identical_models(oracle):
    B, k, V = 66, 5, 512
    g = torch.Generator(device=DEV).manual_seed(1)
    lp = torch.randn((B, k + 1, V), generator=g, device=DEV) * 3
    lq = lp[:, :k].clone()
    tok = torch.randint(0, V, (B, k), generator=g, device=DEV, dtype=torch.int32)
    u = torch.from_numpy(synth.philox_uniforms(1, 1, B, k + 1)[0]).to(DEV)
    bl = (torch.arange(B, device=DEV, dtype=torch.int32) % (k + 1)).contiguous()
    out = _np(binding.polyspec_verify_level(lp, lq, tok, u, 1.0, block_len=bl, want_probs=True))
    ora = oracle.verify_level(lp.cpu(), lq.cpu(), tok.cpu(), u.cpu(), 1.0, block_len=bl.cpu())
    assert (out["accepted_len"] == bl.cpu().numpy()).all()          # p == q accepts everything presented
    counts, bad = H.compare_level_batch(out["accepted_len"], out["next_token"], ora)
    _assert_parity(counts, bad, B * k, "block_len 0..k, p == q")
    # positions beyond block_len report probability 0
    for b in range(B):
        assert (out["p_at_draft"][b, bl[b]:] == 0).all()


def test_level_disjoint_supports_and_masked_vocab(oracle):
    B, k, V = 64, 3, 4096
    g = torch.Generator(device=DEV).manual_seed(2)
    lp = torch.randn((B, k + 1, V), generator=g, device=DEV) * 2
    lq = torch.randn((B, k, V), generator=g, device=DEV) * 2
    lp[:, :, : V // 2] = float("-inf")
    lq[:, :, V // 2:] = float("-inf")
    tok = torch.randint(0, V // 2, (B, k), generator=g, device=DEV, dtype=torch.int32)
    u = torch.from_numpy(synth.philox_uniforms(2, 1, B, k + 1)[0]).to(DEV)
    out = _np(binding.polyspec_verify_level(lp, lq, tok, u, 1.0))
    ora = oracle.verify_level(lp.cpu(), lq.cpu(), tok.cpu(), u.cpu(), 1.0)
    assert (out["accepted_len"] == 0).all() and (out["next_token"] >= V // 2).all()
    counts, bad = H.compare_level_batch(out["accepted_len"], out["next_token"], ora)
    _assert_parity(counts, bad, B, "disjoint supports")


def test_level_unusable_inputs_set_status_and_minus_one(oracle):
    B, k, V = 8, 3, 1024
    g = torch.Generator(device=DEV).manual_seed(3)
    lp = torch.randn((B, k + 1, V), generator=g, device=DEV)
    lq = lp[:, :k].clone() + 0.5 * torch.randn((B, k, V), generator=g, device=DEV)
    tok = torch.randint(0, V, (B, k), generator=g, device=DEV, dtype=torch.int32)
    u = torch.full((B, k + 1), 1e-6, device=DEV)          # tiny uniforms: everything is accepted
    tok[1, 0] = V                                          # token out of range at the first position
    tok[2, 2] = -1
    lp[3, 1, 17] = float("nan")
    lq[4, 0] = float("-inf")                               # a row with no finite logit
    lp[5, k, 5] = float("inf")                             # unusable bonus row
    out = _np(binding.polyspec_verify_level(lp, lq, tok, u, 1.0))
    ora = oracle.verify_level(lp.cpu(), lq.cpu(), tok.cpu(), u.cpu(), 1.0)
    assert out["device_status"][0] == binding.ERR_BAD_INPUT_ON_DEVICE
    for b in range(B):
        if ora["status"][b] != 0:
            assert out["accepted_len"][b] == -1 and out["next_token"][b] == -1, b
        else:
            assert out["accepted_len"][b] == ora["accepted_len"][b] and out["next_token"][b] == ora["next_token"][b], b
    assert sorted(np.nonzero(ora["status"])[0].tolist()) == [1, 2, 3, 4, 5]


def test_outputs_are_deterministic():
    spec = synth.scaled(synth.config("cfg3"), B=8, V=20000)
    d = synth.make_chain(spec, seed=5, device=DEV)
    a = _run_chain(d)
    b = _run_chain(d)
    for key in ("accepted_len", "block_len", "out_tokens", "out_len"):
        assert (a[key] == b[key]).all()


# ------------------------------------------------------------------ chains, reduced sizes
@pytest.mark.parametrize("name,B,V,sigma", [("cfg2", 24, 4096, None), ("cfg3", 16, 10000, None),
                                            ("cfg5", 12, 8200, 0.5), ("cfg5", 12, 24, 2.0)])
def test_chain_reduced_sizes(oracle, name, B, V, sigma):
    spec = synth.scaled(synth.config(name, sigma=sigma), B=B, V=V)
    d = synth.make_chain(spec, seed=7, device=DEV)
    out = _run_chain(d)
    ora = _oracle_chain(oracle, d)
    counts, bad = H.compare_chain(out, ora)
    _assert_parity(counts, bad, B * sum(spec.k), f"{name} reduced B={B} V={V}")
    assert out["device_status"][0] == 0


# ------------------------------------------------------------------ the benchmark configurations at full size
def test_config1_full(oracle):
    spec = synth.config("cfg1")
    for seed in range(8):
        d = synth.make_chain(spec, seed=seed, device=DEV)
        lp, lq = d["models"]
        out = _np(binding.polyspec_verify_level(lp, lq, d["draft_tokens"], d["uniforms"][0], 1.0, want_probs=True))
        ora = oracle.verify_level(lp.cpu(), lq.cpu(), d["draft_tokens"].cpu(), d["uniforms"][0].cpu(), 1.0)
        counts, bad = H.compare_level_batch(out["accepted_len"], out["next_token"], ora)
        assert not bad and counts["exact"] == 1, (seed, counts, bad)
        m = np.isfinite(ora["p_at"])
        np.testing.assert_allclose(out["p_at_draft"][m], ora["p_at"][m], rtol=1e-5)
        np.testing.assert_allclose(out["q_at_draft"][m], ora["q_at"][m], rtol=1e-5)


def test_config2_full(oracle):
    spec = synth.config("cfg2")
    total = {"exact": 0, "tie_accept": 0, "tie_sample": 0, "mismatch": 0, "skipped_after_tie": 0}
    for seed in range(8):
        d = synth.make_chain(spec, seed=seed, device=DEV)
        counts, bad = H.compare_chain(_run_chain(d), _oracle_chain(oracle, d))
        assert not bad, (seed, bad)
        for key in total:
            total[key] += counts[key]
    _assert_parity(total, [], 8 * 17, "cfg2 full, 8 seeds")


def test_config3_full(oracle):
    spec = synth.config("cfg3")
    d = synth.make_chain(spec, seed=0, device=DEV)
    out = _run_chain(d)
    ora = _oracle_chain(oracle, d)
    counts, bad = H.compare_chain(out, ora)
    _assert_parity(counts, bad, 64 * 12, "cfg3 full")
    # bf16 softmax probabilities at the bottom level, via the single-level call on the same rows
    lv = _np(binding.polyspec_verify_level(d["models"][1].contiguous(), d["models"][2], d["draft_tokens"],
                                           d["uniforms"][1, :, :].contiguous(), spec.temperature, want_probs=True))
    for b in (0, 17, 63):
        for j in (0, 5):
            x = int(d["draft_tokens"][b, j])
            P = oracle.softmax_row(d["models"][1][b, j].cpu(), spec.temperature)[x]
            Q = oracle.softmax_row(d["models"][2][b, j].cpu(), spec.temperature)[x]
            assert abs(lv["p_at_draft"][b, j] - P) <= 2e-3 * P and abs(lv["q_at_draft"][b, j] - Q) <= 2e-3 * Q


@pytest.mark.parametrize("sigma", synth.CFG5_SIGMAS)
def test_config5_full_size_sampled_sequences(oracle, sigma):
    """The launch configuration the benchmark times (B=256, V=152064, four models); the oracle checks a
    sample of the sequences one by one, and the whole batch is checked against properties that hold at
    any size: hand-off bookkeeping and the bottom level's closed-form mean acceptance length."""
    spec = synth.config("cfg5", sigma=sigma)
    d = synth.make_chain(spec, seed=int(sigma * 100), device=DEV)
    out = _run_chain(d)
    seqs = [0, 1, 2, 3, 100, 101, 254, 255]
    sub = [m[seqs].cpu() for m in d["models"]]
    ora = oracle.verify_chain(sub, d["k"], d["draft_tokens"][seqs].cpu(), d["uniforms"][:, seqs].cpu().contiguous(),
                              spec.temperature, threads=8)
    gpu_sub = {key: out[key][:, seqs] for key in ("accepted_len", "block_len", "out_tokens", "out_len")}
    counts, bad = H.compare_chain(gpu_sub, ora)
    _assert_parity(counts, bad, len(seqs) * 20, f"cfg5 sigma={sigma} sampled sequences")
    # whole batch: bookkeeping
    k = spec.k
    assert (out["block_len"][2] == k[2]).all()
    assert (out["block_len"][1] == np.minimum(k[1], out["out_len"][2])).all()
    assert (out["block_len"][0] == np.minimum(k[0], out["out_len"][1])).all()
    assert (out["out_len"] == out["accepted_len"] + 1).all()
    assert (out["accepted_len"] <= out["block_len"]).all() and (out["accepted_len"] >= 0).all()
    for l in range(3):
        for b in (5, 77, 200):
            n = out["out_len"][l, b]
            assert (out["out_tokens"][l, b, :n] >= 0).all() and (out["out_tokens"][l, b, n:] == -1).all()
    # whole batch: E[a] at the bottom level = sum_j prod alpha_i, alpha from a float64 softmax on the device
    P = torch.softmax(d["models"][2][:, :k[2]].double(), dim=-1)
    Q = torch.softmax(d["models"][3].double(), dim=-1)
    alpha = torch.minimum(P, Q).sum(-1)
    expect = torch.cumprod(alpha, dim=1).sum(1).cpu().numpy()
    diff = out["accepted_len"][2] - expect
    se = diff.std(ddof=1) / np.sqrt(len(diff))
    assert abs(diff.mean()) < 3 * se + 1e-9, (sigma, diff.mean(), se)
    # ... and its second moment, E[a^2] = sum_j (2j - 1) P(a >= j), which fixes the variance of the acceptance length
    j = torch.arange(1, k[2] + 1, device=alpha.device, dtype=torch.float64)
    expect2 = ((2 * j - 1) * torch.cumprod(alpha, dim=1)).sum(1).cpu().numpy()
    diff2 = out["accepted_len"][2].astype(np.float64) ** 2 - expect2
    se2 = diff2.std(ddof=1) / np.sqrt(len(diff2))
    assert abs(diff2.mean()) < 3 * se2 + 1e-9, (sigma, diff2.mean(), se2)


@pytest.mark.parametrize("seed_index", [0, 1])
@pytest.mark.parametrize("sigma", synth.CFG5_SIGMAS)
def test_config5_full_batch_every_sequence_against_the_oracle(oracle, sigma, seed_index):
    """The launch configuration the benchmark times, all 256 sequences of the batch compared with the oracle one
    by one (every level, every emitted token), for each inter-level noise and two seeds."""
    import os
    spec = synth.config("cfg5", sigma=sigma)
    d = synth.make_chain(spec, seed=7000 + 100 * seed_index + int(sigma * 4), device=DEV)
    out = _run_chain(d)
    cpu_models = _cpu(d["models"])
    ora = oracle.verify_chain(cpu_models, d["k"], d["draft_tokens"].cpu(), d["uniforms"].cpu(), d["temperature"], threads=os.cpu_count() or 8)
    counts, bad = H.compare_chain(out, ora, distance=H.chain_sample_distance(oracle, cpu_models, d["uniforms"].cpu().numpy(), spec.temperature, ora))
    _assert_parity(counts, bad, spec.B * sum(spec.k), f"cfg5 sigma={sigma} seed {seed_index}, whole batch")
    assert out["device_status"][0] == 0
    assert counts["exact"] + counts["tie_accept"] + counts["tie_sample"] + counts["skipped_after_tie"] == spec.B * 3


@pytest.mark.parametrize("sigma", synth.CFG5_SIGMAS)
def test_config5_sixty_four_seeds_acceptance_length_against_the_closed_form(oracle, sigma):
    """64 seeded instances per inter-level noise (16384 sequences): the bottom level's accepted length has mean
    sum_j prod_{i<=j} alpha_i and second moment sum_j (2j-1) prod_{i<=j} alpha_i given the logits, alpha_i = sum_v
    min(P_i, Q_i) (float64 softmax on the device); the sample mean of the difference must vanish within three standard
    errors.  The first eight sequences of every instance are also compared with the oracle token by token."""
    spec = synth.config("cfg5", sigma=sigma)
    k = spec.k
    seqs = list(range(8))
    diffs, diffs2, acc = [], [], [[], [], []]
    total = {"exact": 0, "tie_accept": 0, "tie_sample": 0, "mismatch": 0, "skipped_after_tie": 0}
    j = torch.arange(1, k[2] + 1, device=DEV, dtype=torch.float64)
    for s in range(64):
        d = synth.make_chain(spec, seed=9000 + s, device=DEV)
        out = _run_chain(d)
        assert out["device_status"][0] == 0
        sub = [m[seqs].cpu() for m in d["models"]]
        ora = oracle.verify_chain(sub, d["k"], d["draft_tokens"][seqs].cpu(), d["uniforms"][:, seqs].cpu().contiguous(),
                                  spec.temperature, threads=8)
        counts, bad = H.compare_chain({key: out[key][:, seqs] for key in ("accepted_len", "block_len", "out_tokens", "out_len")}, ora,
                                      distance=H.chain_sample_distance(oracle, sub, d["uniforms"][:, seqs].cpu().numpy(), spec.temperature, ora))
        assert not bad, (sigma, s, bad[:3])
        for key in total:
            total[key] += counts[key]
        P = torch.softmax(d["models"][2][:, :k[2]].double(), dim=-1)
        Q = torch.softmax(d["models"][3].double(), dim=-1)
        surv = torch.cumprod(torch.minimum(P, Q).sum(-1), dim=1)
        del P, Q
        a = out["accepted_len"][2].astype(np.float64)
        diffs.append(a - surv.sum(1).cpu().numpy())
        diffs2.append(a * a - ((2 * j - 1) * surv).sum(1).cpu().numpy())
        for l in range(3):
            acc[l].append(out["accepted_len"][l].astype(np.float64))
        del d
    diff, diff2 = np.concatenate(diffs), np.concatenate(diffs2)
    se, se2 = diff.std(ddof=1) / np.sqrt(len(diff)), diff2.std(ddof=1) / np.sqrt(len(diff2))
    means = [float(np.concatenate(acc[l]).mean()) for l in range(3)]
    var = [float(np.concatenate(acc[l]).var(ddof=1)) for l in range(3)]
    print(f"[cfg5-stats] sigma={sigma}: {len(diff)} sequences; mean accepted_len M3/M2/M1 levels = {means[2]:.4f}/{means[1]:.4f}/{means[0]:.4f}, "
          f"variance {var[2]:.4f}/{var[1]:.4f}/{var[0]:.4f}; bottom level mean - closed form = {diff.mean():+.5f} (se {se:.5f}), "
          f"second moment - closed form = {diff2.mean():+.5f} (se {se2:.5f}); oracle on 8 sequences per instance: {total}")
    assert abs(diff.mean()) < 3 * se + 1e-9, (sigma, diff.mean(), se)
    assert abs(diff2.mean()) < 3 * se2 + 1e-9, (sigma, diff2.mean(), se2)
    assert total["tie_accept"] + total["tie_sample"] <= max(2, 64 * 8 * 20 // 2000)


def test_chain_host_entry_point_matches_device_entry_point():
    spec = synth.scaled(synth.config("cfg5", sigma=1.0), B=16, V=16384)
    d = synth.make_chain(spec, seed=9, device=DEV)
    ref = _run_chain(d)
    models = [m.cpu().pin_memory() for m in d["models"]]
    rows = [m.shape[1] for m in models]
    ws = torch.empty(binding.polyspec_verify_chain_host_workspace(d["k"], rows, spec.B, spec.V, binding.BF16),
                     dtype=torch.uint8, device=DEV)
    out = binding.polyspec_verify_chain_host(models, d["k"], d["draft_tokens"].cpu().pin_memory(),
                                             d["uniforms"].cpu().pin_memory(), spec.temperature, ws)
    torch.cuda.synchronize()
    for key in ("accepted_len", "block_len", "out_tokens", "out_len"):
        assert (out[key].numpy() == ref[key]).all()
    assert out["host_status"][0] == 0


# ------------------------------------------------------------------ limits of the interface
def test_level_with_the_largest_block(oracle):
    """k = POLYSPEC_MAX_K: a close drafter, so long accepted prefixes occur, up to the whole block."""
    B, k, V = 40, binding.MAX_K, 768
    spec = synth.ChainSpec("maxk", 2, B, V, torch.float32, (k,), 1.0, 3.0, (0.15,), False)
    d = synth.make_chain(spec, seed=11, device=DEV)
    lp, lq = d["models"]
    out = _np(binding.polyspec_verify_level(lp, lq, d["draft_tokens"], d["uniforms"][0], 1.0, want_probs=True))
    ora = oracle.verify_level(lp.cpu(), lq.cpu(), d["draft_tokens"].cpu(), d["uniforms"][0].cpu(), 1.0, threads=8)
    counts, bad = H.compare_level_batch(out["accepted_len"], out["next_token"], ora)
    _assert_parity(counts, bad, B * (k + 1), "k = 32")
    assert ora["accepted_len"].max() >= 16 and ora["accepted_len"].min() < ora["accepted_len"].max()


def test_chain_with_the_largest_number_of_models(oracle):
    n = binding.MAX_MODELS
    spec = synth.ChainSpec("max_models", n, 20, 512, torch.bfloat16, (3,) * (n - 1), 0.8, 3.0, (0.4,) * (n - 1), True)
    d = synth.make_chain(spec, seed=12, device=DEV)
    out = _run_chain(d)
    ora = _oracle_chain(oracle, d)
    counts, bad = H.compare_chain(out, ora)
    _assert_parity(counts, bad, 20 * 3 * (n - 1), "8 models")
    assert out["device_status"][0] == 0


def test_level_with_the_largest_vocabulary(oracle):
    """V = 8192 tiles of 256: the most the sampling pass keeps tile sums for; one more tile is refused."""
    V, B, k = 8192 * 256, 2, 1
    spec = synth.ChainSpec("maxv", 2, B, V, torch.bfloat16, (k,), 1.0, 3.0, (1.0,), False)
    d = synth.make_chain(spec, seed=13, device=DEV)
    lp, lq = d["models"]
    out = _np(binding.polyspec_verify_level(lp, lq, d["draft_tokens"], d["uniforms"][0], 1.0))
    ora = oracle.verify_level(lp.cpu(), lq.cpu(), d["draft_tokens"].cpu(), d["uniforms"][0].cpu(), 1.0, threads=2)
    counts, bad = H.compare_level_batch(out["accepted_len"], out["next_token"], ora)
    _assert_parity(counts, bad, B * 2, "V = 2 Mi")
    with pytest.raises(binding.PolyspecError) as err:
        binding.polyspec_verify_level_workspace(B, k, V + 256, binding.BF16)
    assert err.value.status == binding.ERR_UNSUPPORTED


def test_chain_with_empty_blocks_samples_the_bonus_row(oracle):
    """block_len = 0: nothing to test, the token is drawn from row 0 of p (the bonus row of an empty block)."""
    B, k, V = 9, 3, 2048
    g = torch.Generator(device=DEV).manual_seed(14)
    lp = torch.randn((B, k + 1, V), generator=g, device=DEV) * 3
    lq = torch.randn((B, k, V), generator=g, device=DEV) * 3
    tok = torch.randint(0, V, (B, k), generator=g, device=DEV, dtype=torch.int32)
    u = torch.from_numpy(synth.philox_uniforms(14, 1, B, k + 1)[0]).to(DEV)
    bl = torch.zeros(B, dtype=torch.int32, device=DEV)
    out = _np(binding.polyspec_verify_level(lp, lq, tok, u, 1.0, block_len=bl))
    ora = oracle.verify_level(lp.cpu(), lq.cpu(), tok.cpu(), u.cpu(), 1.0, block_len=bl.cpu())
    assert (out["accepted_len"] == 0).all()
    counts, bad = H.compare_level_batch(out["accepted_len"], out["next_token"], ora)
    _assert_parity(counts, bad, B, "block_len = 0")


@pytest.mark.parametrize("B", [1, 2, 37, 75, 149, 300])
def test_chain_batch_sizes_across_the_cluster_thresholds(oracle, B):
    """The walk uses 8, 4, 2 or 1 CTAs per sequence depending on the batch; the results must not depend on it."""
    spec = synth.scaled(synth.config("cfg3"), B=B, V=6144 + 8)
    d = synth.make_chain(spec, seed=15 + B, device=DEV)
    out = _run_chain(d)
    ora = _oracle_chain(oracle, d)
    counts, bad = H.compare_chain(out, ora)
    _assert_parity(counts, bad, B * sum(spec.k), f"cfg3 recipe at B={B}")


def test_halves_of_the_chain_call_equal_the_whole_call():
    spec = synth.scaled(synth.config("cfg5", sigma=0.5), B=10, V=12288)
    d = synth.make_chain(spec, seed=21, device=DEV)
    whole = _run_chain(d)
    call = binding.ChainCall(d["models"], d["k"], d["draft_tokens"], d["uniforms"], d["temperature"])
    call.row_stats()
    halves = _np(call.walk())
    for key in ("accepted_len", "block_len", "out_tokens", "out_len"):
        assert (halves[key] == whole[key]).all()
    again = _np(call.launch())
    for key in ("accepted_len", "block_len", "out_tokens", "out_len"):
        assert (again[key] == whole[key]).all()


@pytest.mark.parametrize("n_models", [2, 3, 4])
def test_committed_tokens_follow_the_target_distribution(n_models):
    """Losslessness, measured on the GPU without the oracle: whatever the drafters are, the first committed token
    is a sample of the target's first row and, given that it was accepted, so is the second of its second row
    (Section 3.1: the verification rule preserves the target distribution).  Every sequence sees the same logits,
    the drafts are drawn from the bottom drafter per sequence and the uniforms are Philox draws, so the committed
    tokens are i.i.d.; chi-square against the float64 softmax."""
    from scipy import stats as sps
    B, V, T = 300_000, 48, 0.8
    k = [3, 4, 5][: n_models - 1]
    g = torch.Generator(device=DEV).manual_seed(11 + n_models)
    rows = [k[l] + 1 for l in range(n_models - 1)] + [k[-1]]
    base = torch.randn((max(rows), V), generator=g, device=DEV) * 2.0
    models = []
    for i in range(n_models):
        one = base[: rows[i]] + (0.8 * i) * torch.randn((rows[i], V), generator=g, device=DEV)
        models.append(one.unsqueeze(0).expand(B, rows[i], V).contiguous())
    q = torch.softmax(models[-1][0].double() / T, dim=-1)
    draft = torch.multinomial(q, B, replacement=True, generator=g).t().contiguous().to(torch.int32)      # [B, k_bottom]
    u = torch.from_numpy(synth.philox_uniforms(77, n_models - 1, B, max(k) + 1)).to(DEV)
    out = _np(binding.polyspec_verify_chain(models, k, draft, u, T))
    assert out["device_status"][0] == 0
    p0 = torch.softmax(models[0][0, 0].double() / T, dim=-1).cpu().numpy()
    first = out["out_tokens"][0, :, 0]
    counts = np.bincount(first, minlength=V).astype(np.float64)
    chi2 = ((counts - B * p0) ** 2 / (B * p0)).sum()
    assert chi2 < sps.chi2.ppf(1 - 1e-6, V - 1), (n_models, chi2)
    # second committed token, for the sequences that committed at least two: a sample of row 1
    two = out["out_len"][0] >= 2
    p1 = torch.softmax(models[0][0, 1].double() / T, dim=-1).cpu().numpy()
    c1 = np.bincount(out["out_tokens"][0, two, 1], minlength=V).astype(np.float64)
    n1 = two.sum()
    assert n1 > B // 20
    chi2 = ((c1 - n1 * p1) ** 2 / (n1 * p1)).sum()
    assert chi2 < sps.chi2.ppf(1 - 1e-6, V - 1), (n_models, "second", chi2)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("T,scale,shift", [(0.05, 6.0, 0.0), (0.3, 40.0, 900.0), (5.0, 0.5, -3000.0), (1.0, 200.0, 0.0)])
def test_level_extreme_temperatures_scales_and_offsets(oracle, dtype, T, scale, shift):
    """Very peaked and very flat rows, and rows carrying a large common offset: the partial normalisers then differ
    by hundreds of powers of two between segments of one row (rebased exactly or dropped to zero), and a common
    offset must change nothing at all."""
    B, k, V = 96, 4, 20480 + 8
    g = torch.Generator(device=DEV).manual_seed(int(T * 100) + int(scale))
    lp = (torch.randn((B, k + 1, V), generator=g, device=DEV) * scale + shift).to(dtype)
    lq = (lp[:, :k].float() + 0.3 * scale * torch.randn((B, k, V), generator=g, device=DEV)).to(dtype)
    probs = torch.softmax(lq.double() / T, dim=-1).float()
    tok = torch.multinomial(probs.reshape(B * k, V), 1, generator=g).reshape(B, k).to(torch.int32)
    u = torch.from_numpy(synth.philox_uniforms(5, 1, B, k + 1)[0]).to(DEV)
    out = _np(binding.polyspec_verify_level(lp, lq, tok, u, T, want_probs=True))
    ora = oracle.verify_level(lp.cpu(), lq.cpu(), tok.cpu(), u.cpu(), T, threads=8)
    assert out["device_status"][0] == 0
    counts, bad = H.compare_level_batch(out["accepted_len"], out["next_token"], ora)
    _assert_parity(counts, bad, B * (k + 1), f"extreme T={T} scale={scale} shift={shift} {dtype}")
    m = np.isfinite(ora["p_at"])
    # |z c| reaches the thousands here: ex2.approx's argument carries 24 bits, so the relative error grows with it
    tol = (1e-5 if dtype == torch.float32 else 2e-3) + 2.0 ** -22 * (abs(shift) + 6 * scale) / T
    np.testing.assert_allclose(out["p_at_draft"][m], ora["p_at"][m], rtol=tol, atol=1e-30)


def test_level_and_chain_random_shapes(oracle):
    """Forty seeded draws of (batch, block lengths, vocabulary, number of models, type, temperature, per-sequence
    block lengths): shapes nobody picked by hand, each against the oracle."""
    rng = np.random.default_rng(20251026)
    total = {"exact": 0, "tie_accept": 0, "tie_sample": 0, "mismatch": 0}
    for case in range(40):
        n_models = int(rng.integers(2, 6))
        B = int(rng.integers(1, 70))
        V = 8 * int(rng.integers(1, 700))
        k = tuple(int(x) for x in rng.integers(1, 13, size=n_models - 1))
        if case % 8 == 0:
            k = k[:-1] + (32,)                                   # the longest block at the bottom now and then
        dtype = torch.float32 if rng.random() < 0.5 else torch.bfloat16
        T = float(rng.choice([0.5, 0.8, 1.0, 1.7]))
        sig = tuple(float(x) for x in rng.uniform(0.3, 2.5, size=n_models - 1))
        spec = synth.ChainSpec(f"rand{case}", n_models, B, V, dtype, k, T, 2.5, sig, bool(rng.random() < 0.5))
        d = synth.make_chain(spec, seed=1000 + case, device=DEV)
        out = _run_chain(d)
        ora = _oracle_chain(oracle, d, threads=8)
        counts, bad = H.compare_chain(out, ora)
        assert not bad, (case, n_models, B, V, k, dtype, T, bad[:3])
        for key in total:
            total[key] += counts[key]
        if n_models == 2:                                        # the single-level call with ragged block lengths
            bl = torch.from_numpy(rng.integers(0, k[0] + 1, size=B).astype(np.int32)).to(DEV)
            lv = _np(binding.polyspec_verify_level(d["models"][0], d["models"][1][:, : k[0]].contiguous(), d["draft_tokens"],
                                                   d["uniforms"][0].contiguous(), T, block_len=bl))
            ol = oracle.verify_level(d["models"][0].cpu(), d["models"][1].cpu(), d["draft_tokens"].cpu(), d["uniforms"][0].cpu(), T,
                                     block_len=bl.cpu())
            c2, bad2 = H.compare_level_batch(lv["accepted_len"], lv["next_token"], ol)
            assert not bad2, (case, B, V, k, bad2[:3])
    print(f"[parity] random shapes: {total}")
    assert total["tie_accept"] + total["tie_sample"] <= 4
