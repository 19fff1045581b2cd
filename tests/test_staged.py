"""Staged verification with a threshold (Section 3.3, Algorithm 1): the host loop of
paper_2510_26527_b200/staged.py, driven here by the CPU oracle (and, in the gpu test, by the CUDA
library on the same inputs).

Pins of the schedule itself, beyond those of the level rule:
  - the committed text keeps the target's distribution although several M_2 rounds are accumulated
    before M_1 looks (Monte Carlo over uniforms and drafts on a tiny vocabulary, 4-sigma bounds);
  - bookkeeping: every M_1 call is presented at least min(mu, what fits) tokens, commits at most one
    more than it was presented, and larger thresholds commit more tokens per M_1 call.
"""
import numpy as np
import pytest
import torch
from scipy.special import softmax as sp_softmax

from paper_2510_26527_b200 import staged, synth


class OracleLevel:
    def __init__(self, oracle, temperature):
        self.oracle, self.T = oracle, temperature

    def level(self, rows_p, rows_q, tokens, uniforms):
        out = self.oracle.verify_level(rows_p.cpu().unsqueeze(0), rows_q.cpu().unsqueeze(0), tokens.cpu().unsqueeze(0),
                                       uniforms.cpu().unsqueeze(0), self.T)
        assert out["status"][0] == 0
        return int(out["accepted_len"][0]), int(out["next_token"][0])


def _models(N, V, seed, s2=0.6, s3=1.2, dtype=torch.float32, device="cpu"):
    g = torch.Generator(device=device).manual_seed(seed)
    M1 = (torch.randn((N, V), generator=g, device=device) * 2.0)
    M2 = M1 + torch.randn((N, V), generator=g, device=device) * s2
    M3 = M1 + torch.randn((N, V), generator=g, device=device) * s3
    return [m.to(dtype).contiguous() for m in (M1, M2, M3)]


def _uniform_tables(seed, rounds, cycles, K):
    u2 = torch.from_numpy(synth.philox_uniforms(seed, 1, rounds, K + 1)[0])
    u1 = torch.from_numpy(synth.philox_uniforms(seed + 1, 1, cycles, staged.MAX_BLOCK + 1)[0])
    return u2, u1


def test_committed_text_keeps_the_target_distribution(oracle):
    V, N, K, mu, T = 6, 48, 3, 5, 1.0
    M1, M2, M3 = _models(N, V, seed=41)
    P1 = sp_softmax(M1.double().numpy() / T, axis=-1)
    Q3 = sp_softmax(M3.double().numpy() / T, axis=-1)
    backend = OracleLevel(oracle, T)
    r = np.random.default_rng(42)
    trials = 6000
    counts = np.zeros((2, V))
    for i in range(trials):
        drafts = torch.tensor([r.choice(V, p=Q3[j]) for j in range(N)], dtype=torch.int32)
        u2, u1 = _uniform_tables(1000 + 2 * i, 16, 4, K)
        res = staged.staged_decode(backend, M1, M2, M3, drafts, u2, u1, K, mu, n_tokens=2)
        counts[0, res.committed[0]] += 1
        counts[1, res.committed[1]] += 1
    for pos in (0, 1):
        freq = counts[pos] / trials
        sigma = np.sqrt(P1[pos] * (1 - P1[pos]) / trials)
        assert (np.abs(freq - P1[pos]) < 4 * sigma + 1e-9).all(), (pos, freq, P1[pos])


def test_bookkeeping_and_effect_of_the_threshold(oracle):
    V, N, K, T = 64, 700, 4, 1.0
    M1, M2, M3 = _models(N, V, seed=43, s2=0.3, s3=0.8)
    Q3 = sp_softmax(M3.double().numpy() / T, axis=-1)
    r = np.random.default_rng(44)
    drafts = torch.tensor([r.choice(V, p=Q3[j]) for j in range(N)], dtype=torch.int32)
    backend = OracleLevel(oracle, T)
    rate = {}
    for mu in (1, 6, 14):
        u2, u1 = _uniform_tables(45, 600, 400, K)
        res = staged.staged_decode(backend, M1, M2, M3, drafts, u2, u1, K, mu, n_tokens=300)
        assert len(res.committed) >= 300 and sum(res.per_cycle) == len(res.committed)
        assert res.m1_calls == len(res.per_cycle) == len(res.presented)
        for m, c in zip(res.presented, res.per_cycle):
            assert min(mu, staged.MAX_BLOCK - K) <= m <= staged.MAX_BLOCK and 1 <= c <= m + 1
        rate[mu] = res.tokens_per_m1_call
    assert rate[1] < rate[6] < rate[14], rate


@pytest.mark.gpu
def test_staged_schedule_on_the_gpu_matches_the_oracle(oracle):
    from paper_2510_26527_b200 import binding, buildlib
    buildlib.build()
    binding.load_library()
    dev = "cuda:0"
    V, N, K, T = 4096, 500, 5, 0.9
    M1, M2, M3 = _models(N, V, seed=46, s2=0.5, s3=1.0, dtype=torch.bfloat16, device=dev)
    g = torch.Generator(device=dev).manual_seed(47)
    drafts = torch.multinomial(torch.softmax(M3.float() / T, dim=-1), 1, generator=g).reshape(N).to(torch.int32)
    for mu in (1, 7, 16):
        u2, u1 = _uniform_tables(48 + mu, 400, 300, K)
        got = staged.staged_decode(staged.GpuLevel(T), M1, M2, M3, drafts, u2.to(dev), u1.to(dev), K, mu, n_tokens=200)
        ref = staged.staged_decode(OracleLevel(oracle, T), M1.cpu(), M2.cpu(), M3.cpu(), drafts.cpu(), u2, u1, K, mu, n_tokens=200)
        assert got.committed == ref.committed and got.presented == ref.presented and got.per_cycle == ref.per_cycle
        assert got.m2_calls == ref.m2_calls
        print(f"[staged] mu={mu}: {got.tokens_per_m1_call:.2f} tokens per M_1 call, {got.m2_calls / got.m1_calls:.2f} M_2 rounds per M_1 call")
