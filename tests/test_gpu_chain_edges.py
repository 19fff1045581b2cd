"""Edge cases of the chain call on the GPU that the parity file does not reach: unusable input that only an upper
level meets, a residual that vanishes in floating point, the largest vocabulary."""
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


def _oracle(oracle, d):
    return oracle.verify_chain([m.cpu() for m in d["models"]], d["k"], d["draft_tokens"].cpu(), d["uniforms"].cpu(), d["temperature"], threads=8)


def test_unusable_row_met_by_an_upper_level_only(oracle):
    """A NaN in M_2's first row: the bottom level (M_3 over M_4) never sees it and reports normally, M_2's level and
    M_1's above it report -1, exactly as the oracle does."""
    spec = synth.scaled(synth.config("cfg5", sigma=0.25), B=6, V=9000)
    d = synth.make_chain(spec, seed=8, device=DEV)
    d["models"][1][2, 0, 100] = float("nan")                     # M_2's first row of sequence 2
    out = _np(binding.polyspec_verify_chain(d["models"], d["k"], d["draft_tokens"], d["uniforms"], d["temperature"]))
    ora = _oracle(oracle, d)
    assert out["device_status"][0] == binding.ERR_BAD_INPUT_ON_DEVICE
    for key in KEYS:
        assert (out[key][:, 2] == ora[key][:, 2]).all(), key
    assert out["accepted_len"][2, 2] >= 0 and out["accepted_len"][1, 2] == -1 and out["accepted_len"][0, 2] == -1
    counts, bad = H.compare_chain(out, ora, seqs=[0, 1, 3, 4, 5])
    assert not bad


def test_residual_that_vanishes_falls_back_to_the_verifier_row(oracle):
    """p == q at the rejected row, the rejection forced by an accept uniform above 1: the residual is 0 everywhere and P
    is sampled instead (the oracle flags the same fall-back)."""
    g = torch.Generator(device=DEV).manual_seed(3)
    for Vv in (16384 + 512, 2048):
        lp = torch.randn((6, 3, Vv), generator=g, device=DEV) * 2
        lq = lp[:, :2].clone()
        tok = torch.randint(0, Vv, (6, 2), generator=g, device=DEV, dtype=torch.int32)
        u = torch.from_numpy(synth.philox_uniforms(4, 1, 6, 3)[0]).to(DEV)
        u[:, 0] = 1.5
        out = _np(binding.polyspec_verify_level(lp, lq, tok, u, 1.0))
        ora = oracle.verify_level(lp.cpu(), lq.cpu(), tok.cpu(), u.cpu(), 1.0)
        assert (ora["fallback"] == 1).all() and (out["accepted_len"] == 0).all()
        assert (out["next_token"] == ora["next_token"]).all(), (Vv, out["next_token"], ora["next_token"])


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_the_largest_vocabulary_the_library_takes(oracle, dtype):
    """V = 8192 tiles of 256 entries, the most the sampling pass keeps tile sums for: three models on two sequences
    against the oracle (both rules), the token drawn from the far end of a row included; eight entries more are
    refused before anything is launched."""
    V, B, k = 8192 * 256, 2, [2, 3]
    g = torch.Generator(device=DEV).manual_seed(91)
    rows = [k[0] + 1, k[1] + 1, k[1]]
    base = torch.randn((B, 4, V), generator=g, device=DEV) * 3.0
    models = []
    for i, r in enumerate(rows):
        m = base[:, :r] if i == 0 else base[:, :r] + torch.randn((B, r, V), generator=g, device=DEV) * 0.7
        models.append(m.to(dtype).contiguous())
    del base
    q = torch.softmax(models[-1].float(), dim=-1)
    drafts = torch.multinomial(q.reshape(-1, V), 1, generator=g).reshape(B, k[1]).to(torch.int32).contiguous()
    del q
    u = torch.from_numpy(synth.philox_uniforms(92, 2, B, max(k) + 1)).to(DEV)
    u[:, 1, max(k)] = 0.99999994                 # sequence 1 samples at the very end of the running sum at both levels
    out = _np(binding.polyspec_verify_chain(models, k, drafts, u, 1.0))
    ora = oracle.verify_chain([m.cpu() for m in models], k, drafts.cpu(), u.cpu(), 1.0, threads=8)
    counts, bad = H.compare_chain(out, ora)
    assert not bad, bad[:2]
    assert out["device_status"][0] == 0
    assert out["out_tokens"][:, 1].max() > V - V // 50          # the late uniform did reach the far end of a row
    got = binding.polyspec_verify_chain_greedy(models, k, drafts)
    torch.cuda.synchronize()
    gra = oracle.verify_chain_greedy([m.cpu() for m in models], k, drafts.cpu(), threads=8)
    for key in KEYS:
        assert (got[key].cpu().numpy() == gra[key]).all(), key
    with pytest.raises(binding.PolyspecError) as e:
        binding.polyspec_verify_chain_workspace(k, rows, B, V + 8, binding._dt(models[0]))
    assert e.value.status == binding.ERR_UNSUPPORTED
