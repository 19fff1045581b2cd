"""Small batches in one launch: polyspec_verify_chain / polyspec_verify_level take a single cluster kernel when a
sequence's rows fit the shared memory of eight CTAs (the paper's setting is batch size 1, Section 4.1).  Its
results must be those of the two launches (polyspec_chain_row_stats + polyspec_chain_walk) bit for bit, and both
are held to the oracle like every other path."""
import numpy as np
import pytest
import torch

from paper_2510_26527_b200 import binding, buildlib, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def lib():
    buildlib.build()
    return binding.load_library()


def _chain(B, V, k, dtype, seed, sigma=1.0, T=1.0):
    g = torch.Generator(device=DEV).manual_seed(seed)
    n = len(k) + 1
    rows = [kk + 1 for kk in k] + [k[-1]]
    base = torch.randn((B, max(rows), V), generator=g, device=DEV) * 3.0
    models = []
    cur = base
    for i in range(n):
        if i:
            cur = cur + torch.randn(cur.shape, generator=g, device=DEV) * sigma
        models.append(cur[:, : rows[i]].to(dtype).contiguous())
    q = torch.softmax(models[-1].float() / T, dim=-1)
    drafts = torch.multinomial(q.reshape(-1, V), 1, generator=g).reshape(B, k[-1]).to(torch.int32).contiguous()
    u = torch.from_numpy(synth.philox_uniforms(seed, len(k), B, max(k) + 1)).to(DEV)
    return models, drafts, u


def _both_paths(models, k, drafts, u, T):
    call = binding.ChainCall(models, k, drafts, u, T)
    one = {n: t.clone() for n, t in call.launch().items()}
    torch.cuda.synchronize()
    for t in call.out.values():
        t.fill_(-7)
    call.device_status.zero_()
    call.row_stats()
    two = {n: t.clone() for n, t in call.walk().items()}
    torch.cuda.synchronize()
    return call, one, two


@pytest.mark.parametrize("B,V,k,dtype", [
    (1, 32000, (4,), torch.float32),            # the two-model workload at batch 1
    (1, 32000, (9, 8), torch.bfloat16),         # the three-model workload at batch 1: 221 KB of rows per CTA
    (2, 32000, (9, 8), torch.bfloat16),
    (16, 32000, (4,), torch.float32),
    (3, 8, (2, 3), torch.float32),              # one vector per row: seven CTAs of the cluster hold nothing
    (5, 2048, (5, 5, 5), torch.bfloat16),       # exactly one segment
    (4, 2056, (3, 2), torch.bfloat16),          # one segment and one vector
    (2, 50264, (3, 2), torch.bfloat16),         # ragged last tile, ragged last segment
    (7, 10000, (20,), torch.bfloat16),          # a long block: 41 rows, three CTAs of the cluster hold nothing
    (1, 151936, (2,), torch.bfloat16),          # a large vocabulary that still fits: 5 rows
])
def test_one_launch_equals_two_launches_and_the_oracle(lib, oracle, B, V, k, dtype):
    T = 0.9
    models, drafts, u = _chain(B, V, list(k), dtype, seed=B * 1000 + V % 977 + len(k))
    call, one, two = _both_paths(models, list(k), drafts, u, T)
    assert call.launches == 1, "this shape is meant to take the cluster kernel"
    for name in ("accepted_len", "block_len", "out_tokens", "out_len"):
        assert torch.equal(one[name], two[name]), name
    assert int(one["device_status"].item()) == 0
    ora = oracle.verify_chain([m.cpu() for m in models], list(k), drafts.cpu(), u.cpu(), T, threads=8)
    counts, bad = H.compare_chain({n: t.cpu().numpy() for n, t in one.items()}, ora)
    assert not bad, bad[:3]
    assert counts["tie_accept"] + counts["tie_sample"] <= 2, counts


def test_level_call_with_block_lengths_probabilities_and_bad_rows(lib):
    """polyspec_verify_level on a small batch goes through the same kernel: per-sequence block lengths, the
    probabilities at the drafted tokens, a NaN row, a token out of range, a row with no finite logit."""
    B, V, k, T = 6, 4096, 5, 1.1
    models, drafts, u = _chain(B, V, [k], torch.float32, seed=5)
    p, q = models
    block_len = torch.tensor([5, 0, 3, 5, 5, 2], dtype=torch.int32, device=DEV)
    p[3, 0, 17] = float("nan")                 # position 0 is always looked at
    drafts[4, 0] = V + 3
    q[5, 0, :] = float("-inf")
    u1 = u[0].contiguous()
    got = binding.polyspec_verify_level(p, q, drafts, u1, T, block_len=block_len, want_probs=True)
    torch.cuda.synchronize()
    # the same call as two launches on the library's static scratch
    ref = {"accepted_len": torch.empty_like(got["accepted_len"]), "next_token": torch.empty_like(got["next_token"]),
           "p_at_draft": torch.empty_like(got["p_at_draft"]), "q_at_draft": torch.empty_like(got["q_at_draft"])}
    binding.polyspec_verify_level_static(p, q, drafts, u1, T, ref, block_len=block_len)
    torch.cuda.synchronize()
    for name in ("accepted_len", "next_token"):
        assert torch.equal(got[name], ref[name]), name
    assert torch.equal(got["p_at_draft"], ref["p_at_draft"]) and torch.equal(got["q_at_draft"], ref["q_at_draft"])
    assert got["accepted_len"][3].item() == -1 and got["accepted_len"][4].item() == -1 and got["accepted_len"][5].item() == -1
    assert got["accepted_len"][1].item() == 0 and got["next_token"][1].item() >= 0
    assert int(got["device_status"].item()) == binding.ERR_BAD_INPUT_ON_DEVICE


def test_one_launch_under_a_cuda_graph_and_on_a_side_stream(lib):
    models, drafts, u = _chain(1, 32000, [9, 8], torch.bfloat16, seed=77)
    s = torch.cuda.Stream()
    call = binding.ChainCall(models, [9, 8], drafts, u, 1.0, stream=s.cuda_stream)
    with torch.cuda.stream(s):
        call.launch()
        s.synchronize()
        want = {n: t.clone() for n, t in call.out.items()}
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            call.launch()
        for t in call.out.values():
            t.fill_(-3)
        g.replay()
        s.synchronize()
    for name in ("accepted_len", "block_len", "out_tokens", "out_len"):
        assert torch.equal(call.out[name], want[name]), name
