"""Staged verification with a threshold (Section 3.3, Algorithm 1).

CPU part: two more pins of the oracle's schedule (oracle/staged.py) beyond the exact enumeration of
tests/test_oracle_staged.py -- the committed text keeps the target's distribution at sizes the enumeration
cannot reach (Monte Carlo), and the threshold does what the section says it is for (larger thresholds commit
more tokens per pass of M_1).

GPU part: the library's batched loop (device-resident bookkeeping kernels + two polyspec_verify_level calls per
iteration, driven by paper_2510_26527_b200/staged.py) against the oracle's plain per-sequence loop, which shares
no code with it: committed text, block presented to every pass of M_1, tokens committed by every pass, rounds of M_2.
"""
import numpy as np
import pytest
import torch
from scipy.special import softmax as sp_softmax

from oracle import staged as ostaged
from paper_2510_26527_b200 import synth

MAXB = ostaged.MAX_BLOCK


def _models(N, V, seed, s2=0.6, s3=1.2, B=None, dtype=torch.float32, device="cpu"):
    g = torch.Generator(device=device).manual_seed(seed)
    shape = (N, V) if B is None else (B, N, V)
    M1 = (torch.randn(shape, generator=g, device=device) * 2.0)
    M2 = M1 + torch.randn(shape, generator=g, device=device) * s2
    M3 = M1 + torch.randn(shape, generator=g, device=device) * s3
    return [m.to(dtype).contiguous() for m in (M1, M2, M3)]


def _uniform_tables(seed, rounds, cycles, K):
    u2 = synth.philox_uniforms(seed, 1, rounds, K + 1)[0]
    u1 = synth.philox_uniforms(seed + 1, 1, cycles, MAXB + 1)[0]
    return u2, u1


def test_committed_text_keeps_the_target_distribution():
    V, N, K, mu, T = 6, 48, 3, 5, 1.0
    M1, M2, M3 = [m.numpy() for m in _models(N, V, seed=41)]
    P1 = sp_softmax(M1.astype(np.float64) / T, axis=-1)
    Q3 = sp_softmax(M3.astype(np.float64) / T, axis=-1)
    r = np.random.default_rng(42)
    trials = 6000
    counts = np.zeros((2, V))
    for i in range(trials):
        drafts = np.array([r.choice(V, p=Q3[j]) for j in range(N)], dtype=np.int32)
        u2, u1 = _uniform_tables(1000 + 2 * i, 16, 4, K)
        res = ostaged.staged_decode(M1, M2, M3, drafts, u2, u1, K, mu, 2, T)
        counts[0, res["committed"][0]] += 1
        counts[1, res["committed"][1]] += 1
    for pos in (0, 1):
        freq = counts[pos] / trials
        sigma = np.sqrt(P1[pos] * (1 - P1[pos]) / trials)
        assert (np.abs(freq - P1[pos]) < 4 * sigma + 1e-9).all(), (pos, freq, P1[pos])


def test_bookkeeping_and_effect_of_the_threshold():
    V, N, K, T = 64, 700, 4, 1.0
    M1, M2, M3 = [m.numpy() for m in _models(N, V, seed=43, s2=0.3, s3=0.8)]
    Q3 = sp_softmax(M3.astype(np.float64) / T, axis=-1)
    r = np.random.default_rng(44)
    drafts = np.array([r.choice(V, p=Q3[j]) for j in range(N)], dtype=np.int32)
    rate = {}
    for mu in (1, 6, 14):
        u2, u1 = _uniform_tables(45, 600, 400, K)
        res = ostaged.staged_decode(M1, M2, M3, drafts, u2, u1, K, mu, 300, T)
        assert len(res["committed"]) >= 300 and sum(res["per_cycle"]) == len(res["committed"])
        assert res["m1_calls"] == len(res["per_cycle"]) == len(res["presented"])
        for m, c in zip(res["presented"], res["per_cycle"]):
            assert min(mu, MAXB - K) <= m <= MAXB and 1 <= c <= m + 1
        rate[mu] = len(res["committed"]) / res["m1_calls"]
    assert rate[1] < rate[6] < rate[14], rate


def _gpu_case(B, V, N, K, T, seed, dtype, R, C):
    dev = "cuda:0"
    M1, M2, M3 = _models(N, V, seed=seed, s2=0.5, s3=1.0, B=B, dtype=dtype, device=dev)
    g = torch.Generator(device=dev).manual_seed(seed + 1)
    q = torch.softmax(M3.float() / T, dim=-1)
    drafts = torch.multinomial(q.reshape(B * N, V), 1, generator=g).reshape(B, N).to(torch.int32).contiguous()
    u2 = torch.from_numpy(synth.philox_uniforms(seed + 2, B, R, K + 1)).to(dev)         # [B, R, K+1]
    u1 = torch.from_numpy(synth.philox_uniforms(seed + 3, B, C, MAXB + 1)).to(dev)      # [B, C, 33]
    return M1, M2, M3, drafts, u2, u1


def _compare_with_oracle(got, inputs, K, mu, n_tokens, T):
    M1, M2, M3, drafts, u2, u1 = [x.cpu() for x in inputs]
    B = M1.shape[0]
    rates = []
    for b in range(B):
        ref = ostaged.staged_decode(M1[b], M2[b], M3[b], drafts[b].numpy(), u2[b].numpy(), u1[b].numpy(), K, mu, n_tokens, T)
        n = len(ref["committed"])
        c = ref["m1_calls"]
        assert int(got["done"][b]) == 1, (b, int(got["done"][b]))
        assert int(got["n_committed"][b]) == n and got["committed"][b, :n].tolist() == ref["committed"], b
        assert (got["committed"][b, n:] == -1).all()
        assert int(got["cycles"][b]) == c and int(got["rounds"][b]) == ref["m2_calls"], b
        assert got["presented"][b, :c].tolist() == ref["presented"] and got["per_cycle"][b, :c].tolist() == ref["per_cycle"], b
        assert int(got["t"][b]) == n and int(got["cnt"][b]) == 0
        rates.append(n / c)
    return float(np.mean(rates))


@pytest.mark.gpu
@pytest.mark.parametrize("mu", [1, 7, 16, 32])
def test_batched_staged_schedule_on_the_gpu_matches_the_oracle(mu):
    from paper_2510_26527_b200 import binding, buildlib, staged
    buildlib.build()
    binding.load_library()
    B, V, N, K, T, n_tokens = 24, 4096, 260, 5, 0.9, 120
    inputs = _gpu_case(B, V, N, K, T, seed=46 + mu, dtype=torch.bfloat16, R=700, C=150)
    run = staged.StagedBatch(*inputs, K, mu, n_tokens, T)
    got = run.run()
    assert int(got["remaining"]) == 0 and int(run.status.item()) == 0
    rate = _compare_with_oracle(got, inputs, K, mu, n_tokens, T)
    # no host read-back per level call: one per mu iterations, and a pass of M_1 comes after at most mu iterations, so the
    # loop reads back no more often than the sequence that needed the most passes made them
    assert got["read_backs"] * mu == got["iterations"] and got["read_backs"] <= int(got["cycles"].max())
    print(f"[staged] mu={mu}: {rate:.2f} tokens per M_1 pass, {float((got['rounds'] / got['cycles']).mean()):.2f} M_2 rounds per pass, "
          f"{got['iterations']} iterations, {got['read_backs']} host read-backs for {B} sequences x {n_tokens} tokens")


@pytest.mark.gpu
def test_batched_staged_schedule_fp32_small_vocabulary_and_ragged_progress():
    """Sequences of one batch drift apart (different acceptance rates per sequence), some finish many iterations
    before others and must then sit still; float32 logits, a vocabulary of one tile, K = 1 and a large K."""
    from paper_2510_26527_b200 import binding, buildlib, staged
    buildlib.build()
    binding.load_library()
    for K, mu, seed in ((1, 3, 5), (12, 20, 6)):
        B, V, N, T, n_tokens = 9, 256, 200, 1.0, 60
        M1, M2, M3, drafts, u2, u1 = _gpu_case(B, V, N, K, T, seed=seed, dtype=torch.float32, R=150, C=100)
        M3[:3] = M2[:3]                      # three sequences whose drafter equals M_2: every round is fully accepted
        q = torch.softmax(M3.float() / T, dim=-1)
        g = torch.Generator(device="cuda:0").manual_seed(seed + 9)
        drafts = torch.multinomial(q.reshape(B * N, V), 1, generator=g).reshape(B, N).to(torch.int32).contiguous()
        inputs = (M1, M2, M3, drafts, u2, u1)
        got = staged.StagedBatch(*inputs, K, mu, n_tokens, T).run()
        _compare_with_oracle(got, inputs, K, mu, n_tokens, T)
        assert got["rounds"][:3].float().mean() < got["rounds"][3:].float().mean() or K == 1


@pytest.mark.gpu
def test_batched_staged_schedule_reports_exhaustion_instead_of_reading_past_the_tables():
    from paper_2510_26527_b200 import binding, buildlib, staged
    buildlib.build()
    binding.load_library()
    B, V, N, K, T, mu = 6, 512, 40, 4, 1.0, 6
    inputs = _gpu_case(B, V, N, K, T, seed=77, dtype=torch.bfloat16, R=60, C=40)
    got = staged.StagedBatch(*inputs, K, mu, 500, T).run()           # 500 tokens do not fit 40 positions
    assert int(got["remaining"]) == 0
    assert (got["done"] == binding.STAGED_EXHAUSTED).all()
    assert (got["t"] + got["cnt"] <= N).all() and (got["n_committed"] == got["t"]).all()
    # what was committed before the tables ran out is still the oracle's text
    M1, M2, M3, drafts, u2, u1 = [x.cpu() for x in inputs]
    for b in range(B):
        n = int(got["n_committed"][b])
        ref = ostaged.staged_decode(M1[b], M2[b], M3[b], drafts[b].numpy(), u2[b].numpy(), u1[b].numpy(), K, mu, max(n, 1), T)
        assert ref["committed"][:n] == got["committed"][b, :n].tolist()


def test_staged_entry_points_reject_bad_arguments():
    from paper_2510_26527_b200 import binding, buildlib
    import ctypes
    buildlib.build()
    lib = binding.load_library()
    fake = 4096                                             # never dereferenced: argument checks come first
    ok = binding.StagedState(4, 3, 5, 8, 100, 10, 10, 64, 20, *([fake] * 11))
    assert lib.polyspec_staged_round_begin(ctypes.byref(ok), None, fake, fake, fake, fake, fake, None) == binding.ERR_INVALID_ARG
    for field, value in (("K", 0), ("K", 32), ("mu", 0), ("mu", 33), ("kcap", 7), ("kcap", 33), ("B", 0), ("cap", 0)):
        bad = binding.StagedState(4, 3, 5, 8, 100, 10, 10, 64, 20, *([fake] * 11))
        setattr(bad, field, value)
        assert lib.polyspec_staged_init(ctypes.byref(bad), None) == binding.ERR_INVALID_ARG, (field, value)
    nul = binding.StagedState(4, 3, 5, 8, 100, 10, 10, 64, 20, *([fake] * 10), None)
    assert lib.polyspec_staged_commit(ctypes.byref(nul), fake, fake, fake, None) == binding.ERR_INVALID_ARG
