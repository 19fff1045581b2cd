"""Greedy matching on the GPU (polyspec_verify_chain_greedy) against the CPU oracle, through the C ABI.

Everything here is integer work decided by comparisons of stored logits, so the bar is bit-exact:
accepted lengths, block lengths, stream lengths and every emitted token, with no tie band.
"""
import numpy as np
import pytest
import torch

from paper_2510_26527_b200 import binding, buildlib, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
KEYS = ("accepted_len", "block_len", "out_len", "out_tokens")


@pytest.fixture(scope="module", autouse=True)
def _lib():
    buildlib.build()
    binding.load_library()
    assert torch.cuda.is_available()


def _run(models, k, draft):
    out = binding.polyspec_verify_chain_greedy(models, k, draft)
    torch.cuda.synchronize()
    return {key: v.cpu().numpy() for key, v in out.items()}


def _greedy_drafts(d, mismatch_rate, seed):
    """Tokens a drafter would hand up: mostly the target's own arg max (so prefixes get accepted), some not."""
    g = torch.Generator(device=DEV).manual_seed(seed)
    kb = d["k"][-1]
    top = d["models"][-2][:, :kb].float().argmax(-1)
    rnd = torch.randint(0, d["models"][0].shape[2], top.shape, generator=g, device=DEV)
    flip = torch.rand(top.shape, generator=g, device=DEV) < mismatch_rate
    return torch.where(flip, rnd, top).to(torch.int32).contiguous()


def _same(got, ora):
    for key in KEYS:
        assert (got[key] == ora[key]).all(), (key, np.argwhere(got[key] != ora[key])[:5])


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V,k,B", [(8, 1, 64), (1000, 3, 128), (4104, 5, 96), (20000, 8, 32)])
def test_level_greedy(oracle, dtype, V, k, B):
    spec = synth.ChainSpec("g", 2, B, V, dtype, (k,), 1.0, 3.0, (0.5,), False)
    d = synth.make_chain(spec, seed=V + k, device=DEV)
    draft = _greedy_drafts(d, 0.2, seed=V)
    got = _run([d["models"][0], None], d["k"], draft)
    ora = oracle.verify_chain_greedy([d["models"][0].cpu(), None], d["k"], draft.cpu(), threads=8)
    _same(got, ora)
    assert got["device_status"][0] == 0
    assert len(set(ora["accepted_len"][0].tolist())) >= min(3, k + 1)


def test_ties_and_rounded_logits(oracle):
    """bf16 logits rounded to few distinct values: many exact ties, the first index must win everywhere."""
    B, k, V = 48, 4, 6000
    g = torch.Generator(device=DEV).manual_seed(5)
    lp = (torch.randn((B, k + 1, V), generator=g, device=DEV) * 2).round().clamp(max=3).to(torch.bfloat16)
    draft = torch.randint(0, V, (B, k), generator=g, device=DEV, dtype=torch.int32)
    ora0 = oracle.verify_chain_greedy([lp.cpu(), None], [k], draft.cpu(), threads=8)
    first_top = ora0["out_tokens"][0, :, 0]            # with a random draft the first emitted token is row 0's arg max
    draft[:, 0] = torch.from_numpy(first_top).to(DEV)   # now position 0 is accepted everywhere
    got = _run([lp, None], [k], draft)
    ora = oracle.verify_chain_greedy([lp.cpu(), None], [k], draft.cpu(), threads=8)
    _same(got, ora)
    assert (ora["accepted_len"][0] >= 1).all()


def test_unusable_inputs(oracle):
    B, k, V = 8, 3, 2048
    g = torch.Generator(device=DEV).manual_seed(6)
    lp = torch.randn((B, k + 1, V), generator=g, device=DEV)
    draft = lp[:, :k].argmax(-1).to(torch.int32)          # everything would be accepted
    lp[1, 0, 100] = float("nan")
    lp[2, k, 7] = float("inf")                            # unusable bonus row
    lp[3, 1] = float("-inf")                              # a row with no finite logit
    lp[4, 2, 9] = -float("nan")                           # a NaN with the sign bit set
    draft = lp[:, :k].nan_to_num(nan=-1e9, posinf=-1e9).argmax(-1).to(torch.int32)
    draft[5, 1] = V                                       # token out of range at position 1
    draft[6, 0] = (draft[6, 0] + 1) % V                   # mismatch at 0: the bad things behind it do not matter
    lp[6, 2, 3] = float("nan")
    got = _run([lp, None], [k], draft)
    ora = oracle.verify_chain_greedy([lp.cpu(), None], [k], draft.cpu())
    assert got["device_status"][0] == binding.ERR_BAD_INPUT_ON_DEVICE
    assert sorted(np.nonzero(ora["status"])[0].tolist()) == [1, 2, 3, 4, 5]
    for b in range(B):
        if ora["status"][b]:
            assert got["accepted_len"][0, b] == -1 and (got["out_tokens"][0, b] == -1).all(), b
        else:
            for key in KEYS:
                assert (got[key][0, b] == ora[key][0, b]).all(), (key, b)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_planted_maxima_at_every_word_position_chunk_and_segment(dtype):
    """The arg max of 2-byte logits is kept on packed words with its position recorded per half, per word and per
    chunk: a unique maximum planted at every kind of position (both halves of every word of a lane's four vectors,
    first and later chunks, first and later segments, the ragged end), the same value planted twice (the first
    must win), +0 against -0, and a maximum equal to the largest finite value.  Row 0's arg max is what the rule
    emits after a mismatch at position 0, so it is read off next to torch's own arg max."""
    V = 3 * 8192 + 1032                                    # three whole segments and a ragged fourth (2-byte logits)
    idx = sorted(set([0, 1, 2, 7, 8, 255, 256, 257, 511, 1023, 1024, 1025, 2047, 2048, 4095, 4096, 8191, 8192, 8193,
                      8192 + 1024 + 37, 2 * 8192 - 1, 2 * 8192, 3 * 8192 + 1031, V - 1, V - 8]
                     + [(j * 2 + h) + 8 * (u * 32 + lane) + 1024 * c for j in range(4) for h in (0, 1)
                        for u in range(4) for lane in (0, 5, 31) for c in (0, 3, 7)]))
    idx = [i for i in idx if i < V]
    B = len(idx) + 6
    g = torch.Generator(device=DEV).manual_seed(12)
    lp = (torch.randn((B, 2, V), generator=g, device=DEV) * 2).clamp(-8, 8)
    for b, i in enumerate(idx):
        lp[b, 0, i] = 16.0                                  # a unique maximum
    n = len(idx)
    lp[n + 0, 0, 4097] = 16.0; lp[n + 0, 0, 20001] = 16.0   # the same value twice: the first wins
    lp[n + 1, 0, 9] = 16.0; lp[n + 1, 0, 8] = 16.0          # twice inside one word
    lp[n + 2, 0] = -1.0; lp[n + 2, 0, 300] = -0.0; lp[n + 2, 0, 77] = 0.0      # +0 and -0 compare equal: index 77
    lp[n + 3, 0] = -1.0; lp[n + 3, 0, 77] = -0.0; lp[n + 3, 0, 300] = 0.0      # ... and the other way round: still 77
    lp[n + 4, 0, 12345] = 3.3895e38                         # the largest finite 2-byte value, not +inf
    lp[n + 5, 0] = float("-inf"); lp[n + 5, 0, V - 3] = -1e30
    lp = lp.to(dtype).contiguous()
    want = lp[:, 0].float().argmax(-1)                      # torch returns the first maximal index too
    assert want[n + 2].item() == 77 and want[n + 3].item() == 77 and want[n + 0].item() == 4097
    draft = ((want + 1) % V).to(torch.int32).reshape(B, 1).contiguous()         # never the arg max: a = 0 everywhere
    got = _run([lp, None], [1], draft)
    assert got["device_status"][0] == 0
    assert (got["accepted_len"][0] == 0).all()
    assert (got["out_tokens"][0, :, 0] == want.cpu().numpy()).all(), np.argwhere(got["out_tokens"][0, :, 0] != want.cpu().numpy())[:8]
    # and with the arg max drafted, everything is accepted and the bonus row's arg max follows
    got = _run([lp, None], [1], want.to(torch.int32).reshape(B, 1).contiguous())
    assert (got["accepted_len"][0] == 1).all()
    assert (got["out_tokens"][0, :, 1] == lp[:, 1].float().argmax(-1).cpu().numpy()).all()


@pytest.mark.parametrize("name,B,V,sigma", [("cfg2", 24, 4096, None), ("cfg3", 16, 10000, None), ("cfg5", 12, 8200, 0.25)])
def test_chain_greedy_reduced(oracle, name, B, V, sigma):
    spec = synth.scaled(synth.config(name, sigma=sigma), B=B, V=V)
    d = synth.make_chain(spec, seed=31, device=DEV)
    draft = _greedy_drafts(d, 0.1, seed=32)
    got = _run(d["models"], d["k"], draft)
    ora = oracle.verify_chain_greedy([m.cpu() for m in d["models"]], d["k"], draft.cpu(), threads=8)
    _same(got, ora)


def test_chain_greedy_config5_full_size(oracle):
    """The four-level workload at full size (B=256, V=152064): sampled sequences against the oracle, the
    whole batch against the property that defines the rule (each level's stream is its verifier's arg max)."""
    spec = synth.config("cfg5", sigma=0.25)
    d = synth.make_chain(spec, seed=33, device=DEV)
    draft = _greedy_drafts(d, 0.05, seed=34)
    got = _run(d["models"], d["k"], draft)
    seqs = [0, 1, 100, 255]
    ora = oracle.verify_chain_greedy([m[seqs].cpu() for m in d["models"]], d["k"], draft[seqs].cpu(), threads=4)
    for key in KEYS:
        assert (got[key][:, seqs] == ora[key]).all(), key
    for l in range(3):
        top = d["models"][l].float().argmax(-1).cpu().numpy()
        n = got["out_len"][l]
        for b in range(spec.B):
            assert (got["out_tokens"][l, b, :n[b]] == top[b, :n[b]]).all(), (l, b)
    assert got["device_status"][0] == 0


@pytest.mark.parametrize("sigma", [0.25, 2.0])
def test_greedy_acceptance_statistics_follow_the_closed_form(sigma):
    """Drafts sampled from the drafter's softmax: a position matches with probability
    gamma_j = q_j(arg max p_j), independently, so E[a] = sum_j prod_{i<=j} gamma_i and
    E[a^2] = sum_j (2j - 1) prod_{i<=j} gamma_i at the bottom level; checked over the whole batch."""
    spec = synth.config("cfg5", sigma=sigma)
    d = synth.make_chain(spec, seed=41, device=DEV)
    got = _run(d["models"], d["k"], d["draft_tokens"])
    kb = spec.k[2]
    top = d["models"][2][:, :kb].float().argmax(-1, keepdim=True)
    Q = torch.softmax(d["models"][3].double() / spec.temperature, dim=-1)
    surv = torch.cumprod(Q.gather(-1, top).squeeze(-1), dim=1)
    j = torch.arange(1, kb + 1, device=surv.device, dtype=torch.float64)
    a = got["accepted_len"][2].astype(np.float64)
    for moment, expect in ((a, surv.sum(1)), (a * a, ((2 * j - 1) * surv).sum(1))):
        diff = moment - expect.cpu().numpy()
        se = diff.std(ddof=1) / np.sqrt(len(diff))
        assert abs(diff.mean()) < 3.5 * se + 1e-9, (sigma, diff.mean(), se)
