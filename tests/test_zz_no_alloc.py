"""polyspec_verify_level_static: the entry point for callers that cannot allocate device memory (a
plugin inside an engine that owns the whole device, code under a fixed memory budget).  It must give
exactly what polyspec_verify_level gives, call after call, although every call reuses one built-in
scratch array that still holds the previous call's partials.  This file is collected last on purpose."""
import pytest
import torch

from paper_2510_26527_b200 import binding, buildlib, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _inputs(seed, B, k, V, dtype):
    spec = synth.ChainSpec("static", 2, B, V, dtype, (k,), 0.8, 3.0, (1.0,), False)
    return synth.make_chain(spec, seed=seed, device=DEV)


def test_static_scratch_entry_point_matches_the_workspace_entry_point_twice_in_a_row(oracle):
    buildlib.build()
    binding.load_library()
    assert binding.polyspec_static_scratch_bytes() == 1 << 20
    # two different problems back to back: the second call finds the first call's partials in the array
    for seed, (B, k, V, dtype) in enumerate([(48, 6, 20000, torch.bfloat16), (7, 3, 4104, torch.float32)]):
        d = _inputs(seed, B, k, V, dtype)
        lp, lq = d["models"]
        u = d["uniforms"][0].contiguous()
        ref = binding.polyspec_verify_level(lp, lq, d["draft_tokens"], u, 0.8, want_probs=True)
        out = {"accepted_len": torch.full((B,), -7, dtype=torch.int32, device=DEV),
               "next_token": torch.full((B,), -7, dtype=torch.int32, device=DEV),
               "p_at_draft": torch.full((B, k), -7.0, device=DEV), "q_at_draft": torch.full((B, k), -7.0, device=DEV)}
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        binding.polyspec_verify_level_static(lp, lq, d["draft_tokens"], u, 0.8, out, device_status=status)
        torch.cuda.synchronize()
        # same kernels, same inputs: integer outputs identical, probabilities within the tests' 1e-5
        assert torch.equal(out["accepted_len"], ref["accepted_len"]) and torch.equal(out["next_token"], ref["next_token"])
        torch.testing.assert_close(out["p_at_draft"], ref["p_at_draft"], rtol=1e-5, atol=0)
        torch.testing.assert_close(out["q_at_draft"], ref["q_at_draft"], rtol=1e-5, atol=0)
        assert int(status.item()) == 0 and (out["accepted_len"] >= 0).all()
        # ... and against the CPU oracle, like every other entry point
        ora = oracle.verify_level(lp.cpu(), lq.cpu(), d["draft_tokens"].cpu(), u.cpu(), 0.8, threads=8)
        assert (out["accepted_len"].cpu().numpy() == ora["accepted_len"]).all()
        assert (out["next_token"].cpu().numpy() == ora["next_token"]).all()


def test_static_scratch_calls_allocate_no_device_memory_and_stale_partials_hide_nothing():
    """What the entry point is for: a caller that may not allocate.  After a first call (which looks up the
    array's address once), further calls must leave the device's free memory exactly as it was.  The last of
    them runs on rows filled with NaN right after a healthy problem of the same shape: were any partial left
    over from the call before it read back, the bad rows would go unnoticed."""
    buildlib.build()
    binding.load_library()
    B, k, V = 32, 4, 16384
    d = _inputs(5, B, k, V, torch.bfloat16)
    lp, lq = d["models"]
    u = d["uniforms"][0].contiguous()
    out = {"accepted_len": torch.empty(B, dtype=torch.int32, device=DEV), "next_token": torch.empty(B, dtype=torch.int32, device=DEV)}
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    bad_p = torch.full_like(lp, float("nan"))
    good = torch.empty_like(out["accepted_len"])
    status_good = torch.empty_like(status)
    binding.polyspec_verify_level_static(lp, lq, d["draft_tokens"], u, 0.8, out, device_status=status)      # warm-up: one-time set-up
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(5):
        binding.polyspec_verify_level_static(lp, lq, d["draft_tokens"], u, 0.8, out, device_status=status)
    good.copy_(out["accepted_len"])          # into memory set aside above: nothing is allocated inside the bracket
    status_good.copy_(status)
    binding.polyspec_verify_level_static(bad_p, lq, d["draft_tokens"], u, 0.8, out, device_status=status)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, (free_before, free_after)
    assert int(status_good.item()) == 0 and (good >= 0).all()
    assert int(status.item()) == binding.ERR_BAD_INPUT_ON_DEVICE
    assert (out["accepted_len"] == -1).all() and (out["next_token"] == -1).all()


def test_static_scratch_entry_point_rejects_problems_beyond_its_limit():
    buildlib.build()
    B, k, V = 4096, 16, 152064                 # needs far more than 1 MiB of partials
    assert binding.polyspec_verify_level_workspace(B, k, V, binding.BF16) > binding.polyspec_static_scratch_bytes()
    fake = torch.zeros(16, dtype=torch.int32, device=DEV)
    st = binding.load_library().polyspec_verify_level_static(
        fake.data_ptr(), fake.data_ptr(), fake.data_ptr(), fake.data_ptr(), None, B, k, V, binding.BF16, 1.0,
        fake.data_ptr(), fake.data_ptr(), None, None, None, None)
    assert st == binding.ERR_SCRATCH_LIMIT
    assert "built-in scratch" in binding.status_string(st)
