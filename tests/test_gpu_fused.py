"""The fused LM-head path on the GPU, through the C ABI, against the CPU oracle.

polyspec_lm_head (the projection alone) is compared with a float64 matmul of the same bf16 inputs:
the tensor core multiplies bf16 exactly and accumulates in fp32 in an unspecified order, so the bound
is the fp32 accumulation error, a small multiple of 2^-24 * sum_d |h_d| |w_d|.

polyspec_verify_from_hidden is compared with the oracle's float64 GEMM + verification.  Logit
differences of ~1e-6 move acceptance ratios and CDF edges by ~1e-5 relative, so besides the 1e-6 tie
band the test counts decisions that differ inside a band of 4x the measured max |dlogit| / T; anything
outside that band is a failure.
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


def _gemm_case(rows, V, d, seed):
    g = torch.Generator(device=DEV).manual_seed(seed)
    h = (torch.randn((rows, d), generator=g, device=DEV) * 1.5).to(torch.bfloat16)
    W = (torch.randn((V, d), generator=g, device=DEV) * 0.05).to(torch.bfloat16)
    return h, W


@pytest.mark.parametrize("rows,V,d", [
    (16, 128, 64),          # one tile, one K block
    (5, 128, 128),          # fewer rows than the MMA's smallest N: zero-filled columns
    (100, 1000, 256),       # ragged vocabulary tile (1000 = 7 * 128 + 104), ragged columns
    (288, 4096, 512),       # two MMAs of N = 144 per K block, single accumulator
    (272, 2048, 192),       # 272 columns are widened to 288
    (300, 2560, 320),       # more rows than one column block: 256-column blocks, two accumulators
    (700, 3200, 128),       # three column blocks, the last one ragged
    (256, 20000, 2048),     # more tiles than SMs: every CTA walks several work items
])
def test_lm_head_matches_float64_matmul(oracle, rows, V, d):
    h, W = _gemm_case(rows, V, d, seed=rows + V + d)
    out, status = binding.polyspec_lm_head(h, W)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle.lm_head_logits(h, W)                                   # float64 on the CPU
    bound = torch.matmul(h.double().abs().cpu(), W.double().abs().cpu().t())   # sum_d |h_d| |w_d|
    err = (out.double().cpu() - ref).abs()
    worst = float((err / bound.clamp(min=1e-30)).max())
    assert worst < 16 * 2.0 ** -24, (rows, V, d, worst)
    # and it is a real product, not zeros
    assert float(ref.abs().max()) > 0.1


def test_lm_head_rejects_bad_arguments():
    h, W = _gemm_case(16, 128, 64, seed=1)
    lib = binding.load_library()
    out = torch.empty((16, 128), device=DEV)
    assert lib.polyspec_lm_head(None, W.data_ptr(), 16, 128, 64, out.data_ptr(), None, None) == binding.ERR_INVALID_ARG
    assert lib.polyspec_lm_head(h.data_ptr(), W.data_ptr(), 16, 128, 40, out.data_ptr(), None, None) == binding.ERR_UNSUPPORTED
    assert lib.polyspec_lm_head(h.data_ptr() + 2, W.data_ptr(), 16, 128, 64, out.data_ptr(), None, None) == binding.ERR_INVALID_ARG


def _fused_compare(oracle, d, band_of_dlogit):
    out = binding.polyspec_verify_from_hidden(d["hidden_p"], d["W_p"], d["hidden_q"], d["W_q"], d["draft_tokens"],
                                              d["uniforms"], d["temperature"], want_probs=True)
    lp, _ = binding.polyspec_lm_head(d["hidden_p"], d["W_p"])
    torch.cuda.synchronize()
    got = {k: v.cpu().numpy() for k, v in out.items()}
    ora = oracle.verify_from_hidden(d["hidden_p"], d["W_p"], d["hidden_q"], d["W_q"], d["draft_tokens"].cpu(),
                                    d["uniforms"].cpu(), d["temperature"], threads=8)
    assert got["device_status"][0] == 0
    # measured logit error of the tensor-core path on this input
    dl = float((lp.double().cpu() - ora["logits_p"]).abs().max())
    assert dl < 1e-4, dl
    band = max(band_of_dlogit(dl), H.TIE_BAND)
    strict, bad = H.compare_level_batch(got["accepted_len"], got["next_token"], ora, band=H.TIE_BAND)
    # every disagreement must be explained by the logit error: an accept test whose uniform lies within
    # 4 dl / T of min(1, P/Q), or a sampling uniform within 8 dl / (T S) of the GPU token's CDF interval
    # (S = residual mass; tokens of negligible mass in between may be skipped, so adjacency is not required)
    T = d["temperature"]
    k = d["draft_tokens"].shape[1]
    u = d["uniforms"].cpu().numpy()
    unexplained = []
    for b, ga, gn, oa, on in bad:
        if ga != oa:
            j = min(ga, oa)
            if not (ora["accept_margin"][b, j] <= band):
                unexplained.append((b, "accept", ga, oa, float(ora["accept_margin"][b, j])))
            continue
        P = H.prob_tables([ora["logits_p"][b, oa].numpy()], T)[0]
        if oa < k:
            Q = H.prob_tables([ora["logits_q"][b, oa].numpy()], T)[0]
            w = np.maximum(P - Q, 0.0)
        else:
            w = P
        dist = H.cdf_distance(w, float(u[b, k]), gn)
        if not (dist <= 2 * band / w.sum()):
            unexplained.append((b, "sample", gn, on, dist, 2 * band / w.sum()))
    print(f"[parity] fused: max |dlogit| {dl:.2e}; 1e-6 band {strict}; explained by the logit error: {len(bad) - len(unexplained)} of {len(bad)}")
    assert not unexplained, unexplained[:5]
    B = len(got["accepted_len"])
    assert strict["mismatch"] <= max(2, B // 16), strict
    m = np.isfinite(ora["p_at"])
    np.testing.assert_allclose(got["p_at_draft"][m], ora["p_at"][m], rtol=2e-4, atol=1e-30)
    np.testing.assert_allclose(got["q_at_draft"][m], ora["q_at"][m], rtol=2e-4, atol=1e-30)
    return got, ora


def test_fused_reduced_size(oracle):
    spec = synth.FusedSpec(B=12, k=5, V=4096, d_p=512, d_q=256)
    d = synth.make_fused(spec, seed=3, device=DEV)
    got, ora = _fused_compare(oracle, d, lambda dl: 4 * dl / spec.temperature)
    assert len(set(ora["accepted_len"].tolist())) >= 3        # the draft tracks the target: several accepted lengths


def test_fused_ragged_vocabulary(oracle):
    """V = 5 * 256 + 40: in the last tile one CTA of the pair sees 40 entries (two of its four lane quarters none),
    the other CTA none at all; their shares of the row statistics must come out empty, not stale."""
    spec = synth.FusedSpec(B=6, k=3, V=1320, d_p=128, d_q=64)
    for seed in (7, 8):                      # a second call reuses whatever the first left in shared memory
        d = synth.make_fused(spec, seed=seed, device=DEV)
        _fused_compare(oracle, d, lambda dl: 4 * dl / spec.temperature)


def test_fused_more_rows_than_one_column_block(oracle):
    """B (k + 1) = 360 hidden rows: two 256-column blocks per vocabulary tile, two alternating accumulators."""
    spec = synth.FusedSpec(B=40, k=8, V=2048, d_p=256, d_q=128)
    d = synth.make_fused(spec, seed=9, device=DEV)
    _fused_compare(oracle, d, lambda dl: 4 * dl / spec.temperature)


def test_fused_config4_full(oracle):
    spec = synth.FusedSpec()
    d = synth.make_fused(spec, seed=0, device=DEV)
    got, ora = _fused_compare(oracle, d, lambda dl: 4 * dl / spec.temperature)
    assert 0.5 < ora["accepted_len"].mean() < spec.k


def test_halves_of_the_fused_call_equal_the_whole_call():
    spec = synth.FusedSpec(B=8, k=4, V=2048, d_p=256, d_q=128)
    d = synth.make_fused(spec, seed=5, device=DEV)
    whole = binding.polyspec_verify_from_hidden(d["hidden_p"], d["W_p"], d["hidden_q"], d["W_q"], d["draft_tokens"],
                                                d["uniforms"], d["temperature"])
    call = binding.FusedCall(d["hidden_p"], d["W_p"], d["hidden_q"], d["W_q"], d["draft_tokens"], d["uniforms"], d["temperature"])
    call.project()
    halves = call.verify()
    torch.cuda.synchronize()
    assert torch.equal(halves["accepted_len"], whole["accepted_len"]) and torch.equal(halves["next_token"], whole["next_token"])
    again = call.launch()
    torch.cuda.synchronize()
    assert torch.equal(again["accepted_len"], whole["accepted_len"]) and torch.equal(again["next_token"], whole["next_token"])
    assert int(call.device_status.item()) == 0


def test_lm_head_random_shapes(oracle):
    """Twenty-four seeded draws of (rows, vocabulary, depth): tile edges nobody picked by hand."""
    rng = np.random.default_rng(2510)
    for case in range(24):
        rows = int(rng.integers(1, 640))
        V = 4 * int(rng.integers(1, 1500))
        d = 64 * int(rng.integers(1, 17))
        h, W = _gemm_case(rows, V, d, seed=9000 + case)
        out, status = binding.polyspec_lm_head(h, W)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        ref = oracle.lm_head_logits(h, W)
        bound = torch.matmul(h.double().abs().cpu(), W.double().abs().cpu().t())
        worst = float(((out.double().cpu() - ref).abs() / bound.clamp(min=1e-30)).max())
        assert worst < 16 * 2.0 ** -24, (case, rows, V, d, worst)


def test_fused_random_shapes(oracle):
    """Twelve seeded draws of the fused call's sizes (batch, block, vocabulary, both depths), each against the oracle."""
    rng = np.random.default_rng(26527)
    for case in range(12):
        k = int(rng.integers(1, 13))
        B = int(rng.integers(1, 1 + 560 // (k + 1)))
        V = 8 * int(rng.integers(16, 700))
        d_q = 64 * int(rng.integers(1, 5))
        d_p = d_q + 64 * int(rng.integers(1, 6))
        spec = synth.FusedSpec(B=B, k=k, V=V, d_p=d_p, d_q=d_q)
        d = synth.make_fused(spec, seed=300 + case, device=DEV)
        print(f"[fused random] case {case}: B={B} k={k} V={V} d_p={d_p} d_q={d_q}")
        _fused_compare(oracle, d, lambda dl: 4 * dl / spec.temperature)
