"""The vocabulary-sharded level on the GPU (polyspec_sharded_level_stats / _decide / _pick), through the C ABI.

One GPU runs every rank's calls one after the other and concatenates the records where the ranks would
all-gather, which computes exactly what n_ranks processes would.  Checked against
  - polyspec_verify_level on the unsharded logits: bit-identical with one rank, and with several ranks
    whenever the slice boundaries fall on the sampling pass's tile boundaries and no sum is near a tie;
  - the CPU oracle on the unsharded logits, with the tie band of the other parity tests.
"""
import numpy as np
import pytest
import torch

from paper_2510_26527_b200 import binding, buildlib, sharded, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _lib():
    buildlib.build()
    binding.load_library()
    assert torch.cuda.is_available()


def _run_sharded(lp, lq, tok, u, T, R, block_len=None, want_probs=False):
    sp, sq = sharded.shard_vocabulary(lp, R), sharded.shard_vocabulary(lq, R)
    calls = [binding.ShardedLevelCall(sp[r], sq[r], tok, u, T, r, R, block_len=block_len, want_probs=want_probs) for r in range(R)]
    accepted, token = sharded.verify_level_sharded_on_one_device(calls)
    torch.cuda.synchronize()
    for a in accepted[1:]:
        assert torch.equal(a, accepted[0])                  # every rank decides the same
    status = max(int(c.device_status[0]) for c in calls)
    return accepted[0].cpu().numpy(), token.cpu().numpy(), status, calls


def _level_inputs(dtype, B, k, V, seed, T=0.9):
    spec = synth.ChainSpec("sharded", 2, B, V, dtype, (k,), T, 2.0, (1.2,), False)
    d = synth.make_chain(spec, seed=seed, device=DEV)
    lp, lq = d["models"]
    return lp, lq, d["draft_tokens"], d["uniforms"][0].contiguous(), T


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V,k", [(64, 3), (1000, 2), (4104, 5), (32000, 4)])
def test_one_rank_is_bit_identical_to_verify_level(dtype, V, k):
    lp, lq, tok, u, T = _level_inputs(dtype, 96, k, V, seed=V + k)
    want = binding.polyspec_verify_level(lp, lq, tok, u, T, want_probs=True)
    torch.cuda.synchronize()
    a, t, status, calls = _run_sharded(lp, lq, tok, u, T, 1, want_probs=True)
    assert status == 0
    assert (a == want["accepted_len"].cpu().numpy()).all()
    assert (t == want["next_token"].cpu().numpy()).all()
    assert torch.equal(calls[0].p_at, want["p_at_draft"]) and torch.equal(calls[0].q_at, want["q_at_draft"])


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("R,V,k", [(2, 1024, 3), (4, 4096, 5), (8, 32768, 4), (2, 1008, 2), (5, 4120, 3), (8, 128256, 6)])
def test_several_ranks_against_the_oracle(oracle, dtype, R, V, k):
    B = 128
    lp, lq, tok, u, T = _level_inputs(dtype, B, k, V, seed=R * 1000 + k)
    a, t, status, _ = _run_sharded(lp, lq, tok, u, T, R)
    assert status == 0
    ora = oracle.verify_level(lp.cpu(), lq.cpu(), tok.cpu(), u.cpu(), T, threads=8)
    counts, bad = H.compare_level_batch(a, t, ora)
    print(f"[parity] sharded R={R} V={V} k={k} {dtype}: {counts}")
    assert not bad, bad[:5]
    assert counts["tie_accept"] + counts["tie_sample"] <= 2
    assert set(np.unique(ora["accepted_len"])) == set(range(k + 1))        # every accepted length occurs
    # and the unsharded library call, which differs from it only by the order of a few additions
    want = binding.polyspec_verify_level(lp, lq, tok, u, T)
    torch.cuda.synchronize()
    same = (a == want["accepted_len"].cpu().numpy()) & (t == want["next_token"].cpu().numpy())
    assert same.sum() >= B - 2


def test_full_size_level_eight_ranks(oracle):
    """The bottom level of the four-model workload at full size (B=256, k=10, V=152064, bf16) over eight ranks:
    sampled sequences against the oracle, the whole batch against the unsharded call."""
    spec = synth.config("cfg5", sigma=1.0)
    d = synth.make_chain(spec, seed=7, device=DEV)
    lp, lq = d["models"][2].contiguous(), d["models"][3].contiguous()
    tok, u, T = d["draft_tokens"], d["uniforms"][2].contiguous(), spec.temperature
    del d
    a, t, status, _ = _run_sharded(lp, lq, tok, u, T, 8)
    assert status == 0
    seqs = [0, 1, 2, 100, 101, 253, 254, 255]
    ora = oracle.verify_level(lp[seqs].cpu(), lq[seqs].cpu(), tok[seqs].cpu(), u[seqs].cpu(), T, threads=8)
    counts, bad = H.compare_level_batch(a[seqs], t[seqs], ora)
    assert not bad, bad[:5]
    want = binding.polyspec_verify_level(lp, lq, tok, u, T)
    torch.cuda.synchronize()
    same = (a == want["accepted_len"].cpu().numpy()) & (t == want["next_token"].cpu().numpy())
    assert same.sum() >= len(a) - 2
    assert (t >= 0).all() and (t < spec.V).all()


def test_block_len_identical_models_and_probabilities(oracle):
    B, k, V, R = 66, 5, 2048, 4
    g = torch.Generator(device=DEV).manual_seed(1)
    lp = torch.randn((B, k + 1, V), generator=g, device=DEV) * 3
    lq = lp[:, :k].clone()
    tok = torch.randint(0, V, (B, k), generator=g, device=DEV, dtype=torch.int32)
    u = torch.from_numpy(synth.philox_uniforms(1, 1, B, k + 1)[0]).to(DEV)
    bl = (torch.arange(B, device=DEV, dtype=torch.int32) % (k + 1)).contiguous()
    a, t, status, calls = _run_sharded(lp, lq, tok, u, 1.0, R, block_len=bl, want_probs=True)
    ora = oracle.verify_level(lp.cpu(), lq.cpu(), tok.cpu(), u.cpu(), 1.0, block_len=bl.cpu())
    assert status == 0 and (a == bl.cpu().numpy()).all()            # p == q accepts everything presented: bonus row sampled
    counts, bad = H.compare_level_batch(a, t, ora)
    assert not bad, bad[:5]
    p_at = calls[0].p_at.cpu().numpy()
    m = np.isfinite(ora["p_at"])
    np.testing.assert_allclose(p_at[m], ora["p_at"][m], rtol=1e-5, atol=1e-30)
    for b in range(B):
        assert (p_at[b, bl[b]:] == 0).all()


def test_mass_on_one_rank_only_and_vanishing_residual(oracle):
    """Disjoint supports put all of p on the last ranks and all of q on the first ones, so the residual lives on
    ranks that own none of the block tokens; equal rows make the residual vanish on every rank, which must fall
    back to sampling P on all of them together."""
    B, k, V, R = 64, 3, 4096, 4
    g = torch.Generator(device=DEV).manual_seed(2)
    lp = torch.randn((B, k + 1, V), generator=g, device=DEV) * 2
    lq = torch.randn((B, k, V), generator=g, device=DEV) * 2
    lp[:, :, : V // 2] = float("-inf")
    lq[:, :, V // 2:] = float("-inf")
    tok = torch.randint(0, V // 2, (B, k), generator=g, device=DEV, dtype=torch.int32)
    u = torch.from_numpy(synth.philox_uniforms(2, 1, B, k + 1)[0]).to(DEV)
    a, t, status, _ = _run_sharded(lp, lq, tok, u, 1.0, R)
    ora = oracle.verify_level(lp.cpu(), lq.cpu(), tok.cpu(), u.cpu(), 1.0)
    assert status == 0 and (a == 0).all() and (t >= V // 2).all()
    counts, bad = H.compare_level_batch(a, t, ora)
    assert not bad, bad[:5]
    # p == q at the rejected row, rejection forced by an accept uniform above 1: residual 0 everywhere -> sample P
    lp2 = torch.randn((B, k + 1, V), generator=g, device=DEV) * 2
    lq2 = lp2[:, :k].clone()
    u2 = u.clone()
    u2[:, 0] = 1.5
    a2, t2, status2, _ = _run_sharded(lp2, lq2, tok, u2, 1.0, R)
    want = binding.polyspec_verify_level(lp2, lq2, tok, u2, 1.0)
    torch.cuda.synchronize()
    assert status2 == 0 and (a2 == 0).all()
    same = (t2 == want["next_token"].cpu().numpy())
    assert same.sum() >= B - 1 and (t2 >= 0).all()


def test_unusable_inputs(oracle):
    B, k, V, R = 8, 3, 1024, 2
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
    a, t, status, _ = _run_sharded(lp, lq, tok, u, 1.0, R)
    ora = oracle.verify_level(lp.cpu(), lq.cpu(), tok.cpu(), u.cpu(), 1.0)
    assert status == binding.ERR_BAD_INPUT_ON_DEVICE
    for b in range(B):
        if ora["status"][b] != 0:
            assert a[b] == -1 and t[b] == -1, b
        else:
            assert a[b] == ora["accepted_len"][b] and t[b] == ora["next_token"][b], b


def test_argument_checks():
    lp = torch.zeros((2, 3, 64), device=DEV)
    lq = torch.zeros((2, 2, 64), device=DEV)
    tok = torch.zeros((2, 2), dtype=torch.int32, device=DEV)
    u = torch.zeros((2, 3), device=DEV)
    call = binding.ShardedLevelCall(lp, lq, tok, u, 1.0, 0, 2)
    with pytest.raises(ValueError):
        call.decide(torch.zeros(call.stats_bytes, dtype=torch.uint8, device=DEV))       # one rank's record, two needed
    with pytest.raises(binding.PolyspecError):
        binding.ShardedLevelCall(lp, lq, tok, u, 1.0, 2, 2).stats()                     # rank out of range
    with pytest.raises(binding.PolyspecError):
        binding.polyspec_sharded_level_sizes(2, 2, 60, binding.F32, 2)                  # slice not a multiple of 8
    with pytest.raises(binding.PolyspecError):
        binding.polyspec_sharded_level_sizes(2, 2, 64, binding.F32, 65)                 # too many ranks


# ------------------------------------------------------------------------------------------------ chains
CHAIN_KEYS = ("accepted_len", "block_len", "out_len", "out_tokens")


def _run_sharded_chain(d, R):
    shards = [sharded.shard_vocabulary(m, R) for m in d["models"]]
    calls = [binding.ShardedChainCall([s[r] for s in shards], d["k"], d["draft_tokens"], d["uniforms"], d["temperature"], r, R)
             for r in range(R)]
    out = sharded.verify_chain_sharded_on_one_device(calls)
    torch.cuda.synchronize()
    for c in calls[1:]:
        for key in CHAIN_KEYS:
            assert torch.equal(c.out[key], out[key]), key            # every rank ends with the same outputs
    status = max(int(c.device_status[0]) for c in calls)
    return {key: out[key].cpu().numpy() for key in CHAIN_KEYS}, status


@pytest.mark.parametrize("name,B,V,sigma", [("cfg1", 40, 4096, None), ("cfg2", 24, 4096, None), ("cfg3", 16, 10000, None),
                                            ("cfg5", 12, 8200, 0.5)])
def test_chain_one_rank_is_bit_identical_to_verify_chain(name, B, V, sigma):
    spec = synth.scaled(synth.config(name, sigma=sigma), B=B, V=V)
    d = synth.make_chain(spec, seed=61, device=DEV)
    want = binding.polyspec_verify_chain(d["models"], d["k"], d["draft_tokens"], d["uniforms"], d["temperature"])
    torch.cuda.synchronize()
    got, status = _run_sharded_chain(d, 1)
    assert status == 0
    for key in CHAIN_KEYS:
        assert (got[key] == want[key].cpu().numpy()).all(), key


@pytest.mark.parametrize("name,B,V,sigma,R", [("cfg2", 24, 4096, None, 2), ("cfg3", 16, 10240, None, 4), ("cfg5", 12, 8192, 0.5, 8),
                                              ("cfg5", 16, 8200, 1.0, 5), ("cfg5", 8, 152064, 0.25, 8)])
def test_chain_several_ranks_against_the_oracle(oracle, name, B, V, sigma, R):
    spec = synth.scaled(synth.config(name, sigma=sigma), B=B, V=V)
    d = synth.make_chain(spec, seed=62, device=DEV)
    got, status = _run_sharded_chain(d, R)
    assert status == 0
    ora = oracle.verify_chain([m.cpu() for m in d["models"]], d["k"], d["draft_tokens"].cpu(), d["uniforms"].cpu(),
                              d["temperature"], threads=8)
    counts, bad = H.compare_chain(got, ora)
    print(f"[parity] sharded chain {name} R={R}: {counts}")
    assert not bad, bad[:5]
    assert counts["tie_accept"] + counts["tie_sample"] <= 2
    assert (got["out_len"] == got["accepted_len"] + 1).all()


def test_chain_unusable_input_below_reports_minus_one_above():
    spec = synth.scaled(synth.config("cfg5", sigma=0.5), B=6, V=4096)
    d = synth.make_chain(spec, seed=63, device=DEV)
    d["draft_tokens"][2, 0] = spec.V                       # out of range at the bottom level
    d["models"][1][4, 0, 7] = float("nan")                 # an unusable row at level 1
    want = binding.polyspec_verify_chain(d["models"], d["k"], d["draft_tokens"], d["uniforms"], d["temperature"])
    torch.cuda.synchronize()
    got, status = _run_sharded_chain(d, 4)
    assert status == binding.ERR_BAD_INPUT_ON_DEVICE
    assert (got["accepted_len"][:, 2] == -1).all() and (got["out_len"][:, 2] == -1).all() and (got["out_tokens"][:, 2] == -1).all()
    assert got["accepted_len"][2, 4] >= 0 and (got["accepted_len"][:2, 4] == -1).all()
    for key in CHAIN_KEYS:
        w = want[key].cpu().numpy()
        assert (got[key][:, [2, 4]] == w[:, [2, 4]]).all(), key          # the same report as the unsharded call


def test_chain_random_shapes_and_rank_counts(oracle):
    """Sixteen seeded draws of (models, batch, blocks, slice size, ranks, type), each against the oracle's chain."""
    rng = np.random.default_rng(4052)
    for case in range(16):
        n_models = int(rng.integers(2, 5))
        R = int(rng.choice([1, 2, 3, 4, 6, 8]))
        B = int(rng.integers(1, 40))
        V = R * 8 * int(rng.integers(1, 300))
        k = tuple(int(x) for x in rng.integers(1, 11, size=n_models - 1))
        dtype = torch.float32 if rng.random() < 0.5 else torch.bfloat16
        sig = tuple(float(x) for x in rng.uniform(0.3, 2.0, size=n_models - 1))
        spec = synth.ChainSpec(f"rs{case}", n_models, B, V, dtype, k, float(rng.choice([0.6, 1.0, 1.5])), 2.5, sig, True)
        d = synth.make_chain(spec, seed=2000 + case, device=DEV)
        got, status = _run_sharded_chain(d, R)
        assert status == 0
        ora = oracle.verify_chain([m.cpu() for m in d["models"]], d["k"], d["draft_tokens"].cpu(), d["uniforms"].cpu(),
                                  d["temperature"], threads=8)
        counts, bad = H.compare_chain(got, ora)
        assert not bad, (case, n_models, R, B, V, k, dtype, bad[:3])
        assert counts["tie_accept"] + counts["tie_sample"] <= 1, (case, counts)
