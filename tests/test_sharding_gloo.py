"""The N > 1 path on CPU: two `gloo` ranks shard a workload the way `bench.py --gpus N` does.

Sequences are independent, so ranks verify disjoint batches with no data-path collective; what the
multi-rank run adds is host logic only: each rank's shard must be a distinct slice of the global
sequence numbering (Philox counters offset by rank * B), and times / work counts are combined with
MAX / SUM.  The verification itself runs here through the CPU oracle, since the product has no CPU path.
"""
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


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from oracle import oracle as orc
    from paper_2510_26527_b200 import synth
    spec = synth.scaled(synth.config("cfg5", sigma=1.0), B=6, V=512)
    d = synth.make_chain(spec, seed=3, device="cpu", batch_offset=rank * spec.B)
    out = orc.verify_chain(d["models"], d["k"], d["draft_tokens"], d["uniforms"], d["temperature"])
    tokens = int(out["block_len"].clip(min=0).sum())
    emitted = int(out["out_len"][0].sum())
    my_ms = 10.0 + 5.0 * rank
    (t_max, t2), (tok_all, em_all) = bench.reduce_over_ranks([my_ms, 1.0], [tokens, emitted], "cpu", world)
    np.save(os.path.join(out_dir, f"u{rank}.npy"), d["uniforms"].numpy())
    np.save(os.path.join(out_dir, f"r{rank}.npy"), np.array([tokens, emitted, t_max, t2, tok_all, em_all]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_and_reduce(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r = [np.load(tmp_path / f"r{i}.npy") for i in range(world)]
    u = [np.load(tmp_path / f"u{i}.npy") for i in range(world)]
    # the reduction: MAX of times, SUM of work, identical on both ranks
    assert r[0][2] == r[1][2] == 15.0 and r[0][3] == r[1][3] == 1.0
    assert r[0][4] == r[1][4] == r[0][0] + r[1][0]
    assert r[0][5] == r[1][5] == r[0][1] + r[1][1]
    # the shards: rank i holds sequences [i*B, (i+1)*B) of one global Philox numbering, so the shards are
    # disjoint draws and together equal the uniforms of one batch of 2B sequences
    sys.path.insert(0, ROOT)
    from paper_2510_26527_b200 import synth
    L, B, slots = u[0].shape
    whole = synth.philox_uniforms(3, L, world * B, slots)
    assert np.array_equal(np.concatenate(u, axis=1), whole)
    assert not np.array_equal(u[0], u[1])
    # every rank did real work
    assert r[0][0] > 0 and r[1][0] > 0


def _bench(*argv, timeout=300):
    import subprocess
    env = dict(os.environ, OMP_NUM_THREADS="1")
    env.pop("WORLD_SIZE", None)
    env.pop("RANK", None)
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *argv], capture_output=True, text=True,
                          timeout=timeout, env=env, cwd=ROOT)


def test_bench_gpus_flag_launches_that_many_ranks():
    """`bench.py --gpus 2` starts two ranks itself (no outer launcher): they rendezvous, reduce times with MAX and
    work with SUM, and rank 0 alone prints the line, with n_gpus = 2.  Run here on `gloo` without any kernel."""
    import json
    res = _bench("--gpus", "2", "--launch-check")
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(l) for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, res.stdout
    assert lines[0] == {"launch_check": True, "n_gpus": 2, "max_ms": 11.0, "summed_work": 300.0}


def test_bench_gpus_flag_without_a_gpu_fails_in_every_rank():
    """No CPU path: without a CUDA device both ranks of `--gpus 2` stop with the library's own error."""
    if torch.cuda.is_available():
        import pytest
        pytest.skip("a CUDA device is present")
    res = _bench("--gpus", "2", "--steps", "1", "--warmup", "1", "--no-workloads")
    assert res.returncode != 0
    assert res.stderr.count("bench.py needs a CUDA device") >= 2, res.stderr[-3000:]


def test_bench_parity_counters_on_the_host():
    """bench.py compares the batch it timed with the oracle and reports counters; the comparison itself is host logic:
    identical outputs are all exact, a changed token away from any CDF edge is a mismatch, a changed accepted length
    whose uniform sits on the threshold is a counted tie, and levels above a tie are not compared."""
    sys.path.insert(0, ROOT)
    import bench
    from oracle import oracle as orc
    from paper_2510_26527_b200 import synth
    spec = synth.scaled(synth.config("cfg5", sigma=0.5), B=5, V=96)
    d = synth.make_chain(spec, seed=11, device="cpu")
    ora = orc.verify_chain(d["models"], d["k"], d["draft_tokens"], d["uniforms"], d["temperature"])
    sample = {"models": d["models"], "uniforms": d["uniforms"], "temperature": d["temperature"]}
    same = {k: ora[k].copy() for k in ("accepted_len", "block_len", "out_tokens", "out_len")}
    c = bench.parity_chain(same, ora, sample)
    assert c["exact"] == c["compared"] == 5 * 3 and c["mismatch"] == 0
    # a different token at the bottom level of sequence 2, nowhere near an edge: a mismatch, and the walk stops there
    wrong = {k: v.copy() for k, v in same.items()}
    a = int(ora["accepted_len"][2, 2])
    wrong["out_tokens"][2, 2, a] = (int(ora["out_tokens"][2, 2, a]) + 17) % 96
    margin_before = ora["sample_info"][2, 2, 0]
    ora["sample_info"][2, 2, 0] = 0.3
    c = bench.parity_chain(wrong, ora, sample)
    assert c["mismatch"] == 1 and c["compared"] == 5 * 3 - 2
    ora["sample_info"][2, 2, 0] = margin_before
    # an accept decision that flips exactly on its threshold: a tie, the two levels above it are skipped
    tie = {k: v.copy() for k, v in same.items()}
    b = 4
    a = int(ora["accepted_len"][2, b])
    j = min(a, spec.k[2] - 1)
    tie["accepted_len"][2, b] = a - 1 if a > 0 else a + 1
    ora["accept_margin"][2, b, min(int(tie["accepted_len"][2, b]), a)] = 1e-9
    c = bench.parity_chain(tie, ora, sample)
    assert c["tie_accept"] == 1 and c["skipped_after_tie"] == 2 and c["mismatch"] == 0
