"""The exchanges of the vocabulary-sharded level on CPU: `gloo` ranks, each holding one slice of the vocabulary,
run `sharded.verify_level_vocab_parallel` (all-gather of stats records, all-gather of mass records, max of the
token).  The product has no CPU path, so the three per-rank calls are played here by a float64 numpy stand-in
that follows the same protocol (records as opaque bytes, rank order, -1 on the ranks that do not hold the
token); what is under test is the host logic around them, and the end result must be what the oracle computes
on the unsharded logits."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


class NumpyShardCall:
    """One rank's three calls, in float64 numpy, on its slice [rank * V_local, (rank + 1) * V_local)."""

    def __init__(self, lp, lq, tok, u, T, rank, n_ranks):
        self.lp, self.lq = lp.double().numpy() / T, lq.double().numpy() / T
        self.tok, self.u = tok.numpy(), u.double().numpy()
        self.rank, self.R = rank, n_ranks
        self.B, self.k = self.tok.shape
        self.Vl = self.lp.shape[2]

    def stats(self):
        rows = np.concatenate([self.lp, self.lq], axis=1)                       # [B, 2k+1, Vl]
        m = rows.max(-1)
        Z = np.exp(rows - m[..., None]).sum(-1)
        at = np.zeros((self.B, self.k, 2))
        x = self.tok - self.rank * self.Vl
        for b in range(self.B):
            for j in range(self.k):
                if 0 <= x[b, j] < self.Vl:
                    at[b, j] = self.lp[b, j, x[b, j]], self.lq[b, j, x[b, j]]
        rec = np.concatenate([m.ravel(), Z.ravel(), at.ravel()])
        return torch.from_numpy(rec).view(torch.uint8)

    def decide(self, records):
        B, k, R = self.B, self.k, self.R
        rec = records.view(torch.float64).numpy().reshape(R, -1)
        n = B * (2 * k + 1)
        m = rec[:, :n].reshape(R, B, 2 * k + 1)
        Z = rec[:, n:2 * n].reshape(R, B, 2 * k + 1)
        at = rec[:, 2 * n:].reshape(R, B, k, 2)
        M = m.max(0)
        Zall = (Z * np.exp(m - M)).sum(0)
        owner = self.tok // self.Vl
        self.a = np.zeros(B, np.int32)
        mass = np.zeros((B, 2))
        self.resid = []
        self.norm = (M, Zall)
        for b in range(B):
            a = k
            for j in range(k):
                zp, zq = at[owner[b, j], b, j]
                P = np.exp(zp - M[b, j]) / Zall[b, j]
                Q = np.exp(zq - M[b, k + 1 + j]) / Zall[b, k + 1 + j]
                if not self.u[b, j] * Q <= P:
                    a = j
                    break
            self.a[b] = a
            P = np.exp(self.lp[b, a] - M[b, a]) / Zall[b, a]
            if a < k:
                Q = np.exp(self.lq[b, a] - M[b, k + 1 + a]) / Zall[b, k + 1 + a]
                w = np.maximum(0.0, P - Q)
            else:
                w = P
            if a < k and not w.sum() > 0:
                mass[b] = 0.0, P.sum()
                w = P
            else:
                mass[b] = w.sum(), 0.0
            self.resid.append(w)
        return torch.from_numpy(self.a.copy()), torch.from_numpy(mass.ravel()).view(torch.uint8)

    def pick(self, masses):
        ms = masses.view(torch.float64).numpy().reshape(self.R, self.B, 2)
        out = np.full(self.B, -1, np.int32)
        for b in range(self.B):
            col = 0 if (ms[:, b, 0].sum() > 0 or self.a[b] == self.k) else 1
            share = ms[:, b, col]
            target = self.u[b, self.k] * share.sum()
            cum = np.concatenate([[0.0], np.cumsum(share)])
            hit = np.nonzero(cum[1:] > target)[0]
            owner = hit[0] if len(hit) else np.nonzero(share > 0)[0][-1]
            if owner == self.rank:
                c = cum[owner] + np.cumsum(self.resid[b])
                v = np.nonzero(c > target)[0]
                out[b] = self.rank * self.Vl + (v[0] if len(v) else np.nonzero(self.resid[b] > 0)[0][-1])
        return torch.from_numpy(out)


class NumpyChainCall:
    """The chain calls of one rank in float64 numpy: stats once, then gather / decide / pick / handoff per level."""

    def __init__(self, models, k, tok, u, T, rank, n_ranks):
        self.z = [m.double().numpy() / T for m in models]
        self.k, self.L = list(k), len(models) - 1
        self.kmax = max(self.k)
        self.u = u.double().numpy()
        self.rank, self.R = rank, n_ranks
        self.B = tok.shape[0]
        self.Vl = self.z[0].shape[2]
        self.block = np.full((self.B, self.kmax + 1), -1, np.int64)
        self.block[:, : self.k[-1]] = tok.numpy()
        self.block_len = np.full(self.B, self.k[-1], np.int64)
        shape = (self.L, self.B)
        self.out = {"accepted_len": np.full(shape, -9, np.int32), "block_len": np.full(shape, -9, np.int32),
                    "out_len": np.full(shape, -9, np.int32), "out_tokens": np.full(shape + (self.kmax + 1,), -9, np.int32)}

    def stats(self):
        recs = []
        for z in self.z:
            m = z.max(-1)
            recs += [m.ravel(), np.exp(z - m[..., None]).sum(-1).ravel()]
        return torch.from_numpy(np.concatenate(recs)).view(torch.uint8)

    def _norms(self, stats, i):
        """(max, sum) of model i's rows over the whole vocabulary, [B, rows]."""
        rec = stats.view(torch.float64).numpy().reshape(self.R, -1)
        off = sum(2 * self.z[j].shape[0] * self.z[j].shape[1] for j in range(i))
        n = self.z[i].shape[0] * self.z[i].shape[1]
        m = rec[:, off:off + n].reshape(self.R, *self.z[i].shape[:2])
        Z = rec[:, off + n:off + 2 * n].reshape(self.R, *self.z[i].shape[:2])
        M = m.max(0)
        return M, (Z * np.exp(m - M)).sum(0)

    def gather(self, level):
        at = np.zeros((self.B, self.kmax + 1, 2))
        x = self.block - self.rank * self.Vl
        for b in range(self.B):
            for j in range(min(self.k[level], self.block_len[b])):
                if 0 <= x[b, j] < self.Vl:
                    at[b, j] = self.z[level][b, j, x[b, j]], self.z[level + 1][b, j, x[b, j]]
        return torch.from_numpy(at.ravel()).view(torch.uint8)

    def decide(self, level, stats, gathers):
        at = gathers.view(torch.float64).numpy().reshape(self.R, self.B, self.kmax + 1, 2)
        (Mp, Zp), (Mq, Zq) = self._norms(stats, level), self._norms(stats, level + 1)
        owner = np.clip(self.block // self.Vl, 0, self.R - 1)
        mass = np.zeros((self.B, 2))
        self.resid, self.a = [], np.zeros(self.B, np.int64)
        for b in range(self.B):
            m = min(self.k[level], self.block_len[b])
            a = m
            for j in range(m):
                zp, zq = at[owner[b, j], b, j]
                P = np.exp(zp - Mp[b, j]) / Zp[b, j]
                Q = np.exp(zq - Mq[b, j]) / Zq[b, j]
                if not self.u[level, b, j] * Q <= P:
                    a = j
                    break
            self.a[b] = a
            self.out["accepted_len"][level, b], self.out["block_len"][level, b] = a, m
            P = np.exp(self.z[level][b, a] - Mp[b, a]) / Zp[b, a]
            w = np.maximum(0.0, P - np.exp(self.z[level + 1][b, a] - Mq[b, a]) / Zq[b, a]) if a < m else P
            self.bonus = getattr(self, "bonus", {})
            self.bonus[b] = a == m
            if a < m and not w.sum() > 0:
                mass[b] = 0.0, P.sum()
                w = P
            else:
                mass[b] = w.sum(), 0.0
            self.resid.append(w)
        return torch.from_numpy(mass.ravel()).view(torch.uint8)

    def pick(self, level, masses):
        ms = masses.view(torch.float64).numpy().reshape(self.R, self.B, 2)
        out = np.full(self.B, -1, np.int32)
        for b in range(self.B):
            col = 0 if (ms[:, b, 0].sum() > 0 or self.bonus[b]) else 1
            share = ms[:, b, col]
            target = self.u[level, b, self.kmax] * share.sum()
            cum = np.concatenate([[0.0], np.cumsum(share)])
            hit = np.nonzero(cum[1:] > target)[0]
            owner = hit[0] if len(hit) else np.nonzero(share > 0)[0][-1]
            if owner == self.rank:
                c = cum[owner] + np.cumsum(self.resid[b])
                v = np.nonzero(c > target)[0]
                out[b] = self.rank * self.Vl + (v[0] if len(v) else np.nonzero(self.resid[b] > 0)[0][-1])
        return torch.from_numpy(out)

    def handoff(self, level, token):
        t = token.numpy()
        for b in range(self.B):
            a = self.a[b]
            self.block[b, a] = t[b]
            self.block_len[b] = a + 1
            self.out["out_len"][level, b] = a + 1
            self.out["out_tokens"][level, b] = -1
            self.out["out_tokens"][level, b, : a + 1] = self.block[b, : a + 1]


def _chain_worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2510_26527_b200 import sharded, synth
    spec = synth.ChainSpec("sharded", 3, 40, 64 * world, torch.float32, (3, 4), 0.8, 2.0, (0.8, 0.8), True)
    d = synth.make_chain(spec, seed=6, device="cpu")
    slices = [sharded.shard_vocabulary(m, world)[rank] for m in d["models"]]
    call = NumpyChainCall(slices, d["k"], d["draft_tokens"], d["uniforms"], spec.temperature, rank, world)
    out = sharded.verify_chain_vocab_parallel(call)
    np.savez(os.path.join(out_dir, f"c{rank}.npz"), **out)
    dist.barrier()
    dist.destroy_process_group()


def test_chain_two_gloo_ranks(tmp_path):
    world = 2
    mp.spawn(_chain_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    sys.path.insert(0, ROOT)
    from oracle import oracle as orc
    from paper_2510_26527_b200 import synth
    spec = synth.ChainSpec("sharded", 3, 40, 64 * world, torch.float32, (3, 4), 0.8, 2.0, (0.8, 0.8), True)
    d = synth.make_chain(spec, seed=6, device="cpu")
    ora = orc.verify_chain(d["models"], d["k"], d["draft_tokens"], d["uniforms"], spec.temperature)
    got = [np.load(tmp_path / f"c{r}.npz") for r in range(world)]
    for key in ("accepted_len", "block_len", "out_len", "out_tokens"):
        assert np.array_equal(got[0][key], got[1][key]), key
        assert np.array_equal(got[0][key], ora[key]), key
    assert len(set(got[0]["accepted_len"].ravel().tolist())) >= 3


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2510_26527_b200 import sharded, synth
    spec = synth.ChainSpec("sharded", 2, 48, 96 * world, torch.float32, (4,), 0.8, 2.0, (1.0,), False)
    d = synth.make_chain(spec, seed=5, device="cpu")                 # the same full problem on every rank ...
    lp, lq = d["models"]
    sp, sq = sharded.shard_vocabulary(lp, world), sharded.shard_vocabulary(lq, world)
    call = NumpyShardCall(sp[rank], sq[rank], d["draft_tokens"], d["uniforms"][0], spec.temperature, rank, world)   # ... of which it keeps its slice
    accepted, token = sharded.verify_level_vocab_parallel(call)
    np.save(os.path.join(out_dir, f"a{rank}.npy"), accepted.numpy())
    np.save(os.path.join(out_dir, f"t{rank}.npy"), token.numpy())
    dist.barrier()
    dist.destroy_process_group()


def _check(tmp_path, world):
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    sys.path.insert(0, ROOT)
    from oracle import oracle as orc
    from paper_2510_26527_b200 import synth
    spec = synth.ChainSpec("sharded", 2, 48, 96 * world, torch.float32, (4,), 0.8, 2.0, (1.0,), False)
    d = synth.make_chain(spec, seed=5, device="cpu")
    ora = orc.verify_level(d["models"][0], d["models"][1], d["draft_tokens"], d["uniforms"][0], spec.temperature)
    a = [np.load(tmp_path / f"a{r}.npy") for r in range(world)]
    t = [np.load(tmp_path / f"t{r}.npy") for r in range(world)]
    for r in range(1, world):
        assert np.array_equal(a[r], a[0]) and np.array_equal(t[r], t[0])       # every rank ends with the same answer
    assert np.array_equal(a[0], ora["accepted_len"])
    assert np.array_equal(t[0], ora["next_token"])
    assert len(set(a[0].tolist())) >= 3 and (t[0] >= 0).all()


def test_two_gloo_ranks(tmp_path):
    _check(tmp_path, 2)


def test_three_gloo_ranks(tmp_path):
    _check(tmp_path, 3)
