"""Staged verification with a threshold (Section 3.3, "Staged Verification"; Algorithm 1) for a batch of
sequences and three models, driven from Python with all state on the device.

Algorithm 1: M_3 drafts K tokens, M_2 verifies them, and what M_2 hands on is accumulated; once at least
``mu`` tokens have accumulated, M_1 verifies the accumulated block in one pass, the verified part is
committed and t advances.  One iteration of that loop, for every sequence of the batch at once, is

    polyspec_staged_round_begin -> [model forwards] -> polyspec_verify_level (M_2 over M_3's drafts)
    -> polyspec_staged_accumulate -> [model forward] -> polyspec_verify_level (M_1 over the accumulated
    block, block_len = 0 for the sequences still below the threshold) -> polyspec_staged_commit

and nothing in it comes back to the host: the loop reads one device counter (sequences still running) once
every ``mu`` iterations, which is at most once per pass of M_1 for any sequence.  All verification and all
bookkeeping run in the library's kernels; this module only sequences the calls and stands in for the model
forwards.

The stand-in: logits are indexed by position (row i of every model scores position i, whatever the tokens
before it), so "running M_2 on positions s .. s+K" is a gather of rows s .. s+K of its table, done here with
torch indexing on the device positions the library hands out.  That makes the whole schedule runnable and
measurable on synthetic logits: tokens committed per M_1 pass as a function of mu.
"""
from __future__ import annotations

import ctypes
from typing import Dict

import torch

from . import binding

MAX_BLOCK = binding.MAX_K


class StagedBatch:
    """Device state of Algorithm 1's loop for B sequences, and the loop itself.

    M1, M2, M3   [B, N, V] logits by position (bf16 or fp32, CUDA)
    drafts       [B, N] int32: the token M_3 proposes at each position
    u2           [B, R, K+1] float32: row r serves a sequence's r-th M_2 round
    u1           [B, C, MAX_BLOCK+1] float32: row c serves its c-th M_1 pass (slots 0..m-1 accept tests, slot MAX_BLOCK sampling)
    """

    def __init__(self, M1, M2, M3, drafts, u2, u1, K: int, mu: int, n_tokens: int, temperature: float):
        self.lib = binding.load_library()
        for t in (M1, M2, M3, drafts, u2, u1):
            if not t.is_cuda or not t.is_contiguous():
                raise ValueError("StagedBatch takes contiguous CUDA tensors")
        self.M1, self.M2, self.M3, self.drafts, self.u2, self.u1 = M1, M2, M3, drafts, u2, u1
        B, N, V = M1.shape
        if tuple(u2.shape[::2]) != (B, K + 1) or tuple(u1.shape[::2]) != (B, MAX_BLOCK + 1) or tuple(drafts.shape) != (B, N):
            raise ValueError("shapes must be drafts [B,N], u2 [B,R,K+1], u1 [B,C,MAX_BLOCK+1]")
        self.B, self.N, self.V, self.K, self.mu = B, N, V, int(K), int(mu)
        self.kcap = min(MAX_BLOCK, self.mu + self.K)
        self.R, self.C = int(u2.shape[1]), int(u1.shape[1])
        self.n_tokens = int(n_tokens)
        self.cap = self.n_tokens + MAX_BLOCK + 1
        self.temperature = float(temperature)
        dev = M1.device
        i32 = lambda *shape: torch.empty(shape, dtype=torch.int32, device=dev)
        self.state = {name: i32(B) for name in ("t", "cnt", "rounds", "cycles", "n_committed", "done")}
        self.state.update(accepted=i32(B, MAX_BLOCK), committed=i32(B, self.cap), presented=i32(B, self.C),
                          per_cycle=i32(B, self.C), remaining=i32(1))
        self.cstate = binding.StagedState(B, self.K, self.mu, self.kcap, N, self.R, self.C, self.cap, self.n_tokens,
                                          *[self.state[n].data_ptr() for n in binding.STAGED_ARRAYS])
        # inputs and outputs of the two level calls of an iteration, allocated once
        self.pos2, self.block_len2, self.tokens2 = i32(B), i32(B), i32(B, self.K)
        self.uniforms2 = torch.empty((B, self.K + 1), dtype=torch.float32, device=dev)
        self.pos1, self.block_len1, self.tokens1 = i32(B), i32(B), i32(B, self.kcap)
        self.uniforms1 = torch.empty((B, self.kcap + 1), dtype=torch.float32, device=dev)
        self.out2 = {"accepted_len": i32(B), "next_token": i32(B)}
        self.out1 = {"accepted_len": i32(B), "next_token": i32(B)}
        dt = binding._dt(M1)
        self.ws2 = binding._workspace(binding.polyspec_verify_level_workspace(B, self.K, V, dt), dev)
        self.ws1 = binding._workspace(binding.polyspec_verify_level_workspace(B, self.kcap, V, dt), dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self._b = torch.arange(B, device=dev).unsqueeze(1)
        self._ar2 = torch.arange(self.K + 1, device=dev).unsqueeze(0)
        self._ar1 = torch.arange(self.kcap + 1, device=dev).unsqueeze(0)
        self.iterations = 0
        self.read_backs = 0
        self._check(self.lib.polyspec_staged_init(ctypes.byref(self.cstate), binding._stream(None)), "polyspec_staged_init")

    @staticmethod
    def _check(st, where):
        if st != binding.OK:
            raise binding.PolyspecError(st, where)

    def _forward(self, table, pos, ar):
        """Stand-in for a model forward: the rows of a position-indexed logits table from `pos` on, per sequence."""
        idx = (pos.long().unsqueeze(1) + ar).clamp_(max=self.N - 1)
        return table[self._b, idx]

    def iteration(self):
        """One pass through the body of Algorithm 1's loop for every sequence; enqueues only."""
        lib, s, p, q = self.lib, ctypes.byref(self.cstate), binding._ptr, binding._stream(None)
        self._check(lib.polyspec_staged_round_begin(s, p(self.drafts), p(self.u2), p(self.pos2), p(self.tokens2), p(self.uniforms2),
                                                    p(self.block_len2), q), "polyspec_staged_round_begin")
        rows_p = self._forward(self.M2, self.pos2, self._ar2)
        rows_q = self._forward(self.M3, self.pos2, self._ar2[:, : self.K])
        binding.polyspec_verify_level(rows_p, rows_q, self.tokens2, self.uniforms2, self.temperature, block_len=self.block_len2,
                                      workspace=self.ws2, out=self.out2, device_status=self.status)
        self._check(lib.polyspec_staged_accumulate(s, p(self.tokens2), p(self.block_len2), p(self.out2["accepted_len"]),
                                                   p(self.out2["next_token"]), p(self.u1), p(self.pos1), p(self.tokens1),
                                                   p(self.uniforms1), p(self.block_len1), q), "polyspec_staged_accumulate")
        rows_p = self._forward(self.M1, self.pos1, self._ar1)
        rows_q = self._forward(self.M2, self.pos1, self._ar1[:, : self.kcap])
        binding.polyspec_verify_level(rows_p, rows_q, self.tokens1, self.uniforms1, self.temperature, block_len=self.block_len1,
                                      workspace=self.ws1, out=self.out1, device_status=self.status)
        self._check(lib.polyspec_staged_commit(s, p(self.block_len1), p(self.out1["accepted_len"]), p(self.out1["next_token"]), q),
                    "polyspec_staged_commit")
        self.iterations += 1

    def run(self, max_iterations: int = 100000) -> Dict[str, torch.Tensor]:
        """Iterate until every sequence has committed n_tokens (or ran out of positions / uniforms)."""
        while self.iterations < max_iterations:
            for _ in range(self.mu):
                self.iteration()
            self.read_backs += 1
            if int(self.state["remaining"].item()) == 0:            # the loop's only read-back
                break
        return self.results()

    def results(self) -> Dict[str, torch.Tensor]:
        torch.cuda.synchronize()
        out = {k: v.cpu() for k, v in self.state.items()}
        out["iterations"], out["read_backs"] = self.iterations, self.read_backs
        return out


def staged_decode_batch(M1, M2, M3, drafts, u2, u1, K, mu, n_tokens, temperature) -> Dict[str, torch.Tensor]:
    """Algorithm 1 from position 0 for every sequence of the batch; see StagedBatch."""
    return StagedBatch(M1, M2, M3, drafts, u2, u1, K, mu, n_tokens, temperature).run()
