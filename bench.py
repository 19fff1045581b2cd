#!/usr/bin/env python
"""Benchmark of the chained verification step (libpolyspec) on synthetic logits.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5|cfg3|cfg2|cfg1|cfg4] [--impl reference]

One step = one pass of the whole hot path (the temperature-softmax normaliser of every logits row of
every model, accept tests, first rejection, replacement-or-bonus sampling and hand-off for every level)
over one batch that is already resident in HBM.  The headline workload is the largest logits-path
configuration, the four-level chain (B=256 per GPU, V=152064, bf16, k=(10,6,4) bottom-up, 2.57 GB of
logits per call -- larger than L2, so nothing is served from cache between steps).  `--workload cfg4` is
the fused path (hidden states -> LM-head projections on the tensor cores -> verification); its roofline
object is the tensor one.

Prints ONE JSON line (rank 0).  A default run (one GPU, headline workload) also measures the four other
configurations for a fixed number of steps each and embeds their records under "workloads"; every record
carries the parity counters of its timed batch against the CPU oracle.  `--gpus N` launches N ranks (one
per GPU, independent replicas) unless a launcher already did.  `--impl reference` times the CPU oracle
as it stands on the host cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2510_26527_b200 import synth  # noqa: E402

METRIC = "verified_draft_tokens_per_s"
UNIT = "tokens/s"
TIE_BAND = 1e-6

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the kernel that streams the logits, from the
# ncu capture summarised under profiles/ (bytes per logits byte processed, measured on a smaller case of
# the same kernel and scaled by the bytes one launch processes).  None once the kernel has changed since.
STATS_TRAFFIC_PER_LOGIT_BYTE = 1.0116     # profiles/stats_kernel_bf16_cfg3_ncu_full.md: (328.350 + 3.80) MB moved for 328.340 MB of logits
# the same counters per launch of the LM-head kernel on the fused workload
# (profiles/lmhead_kernel_cfg4_ncu.md: 402.98 MB read + 53.81 MB written)
LMHEAD_TRAFFIC_BYTES = 456789504


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            pk = json.load(f)
        return {"hbm_gbs": float(pk["hbm_gbs"]), "bf16_tflops": float(pk["bf16_tflops"]),
                "bf16_tflops_sustained": float(pk.get("bf16_tflops_sustained", pk["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def copy_probe_gbs(dev, nbytes=1 << 30, iters=20):
    """Device-to-device copy bandwidth of the GPU this run landed on (bytes read + bytes written per second).

    Context for the roofline fraction only: boxes of one pool differ by several per cent, and the stored
    peak was measured on one of them.  Taken outside the timed region."""
    src = torch.empty(nbytes, dtype=torch.uint8, device=dev).fill_(1)
    dst = torch.empty_like(src)
    for _ in range(3):
        dst.copy_(src)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(iters):
        dst.copy_(src)
    e1.record()
    torch.cuda.synchronize()
    return 2.0 * nbytes * iters / (e0.elapsed_time(e1) * 1e-3) / 1e9


def copy_probe_sustained_gbs(dev, nbytes=1 << 30, seconds=0.5):
    """The same copy kept up for about as long as the timed region: (bandwidth over its first tenth, over its last tenth).

    A board that streams for tenths of a second settles at a lower bandwidth than it shows in a burst; a kernel timed
    over a thousand steps is mostly in that state, and this is the copy in the same state."""
    src = torch.empty(nbytes, dtype=torch.uint8, device=dev).fill_(1)
    dst = torch.empty_like(src)
    iters = max(100, int(seconds / (2.0 * nbytes / 6.0e12)) // 10 * 10)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(11)]
    torch.cuda.synchronize()
    for seg in range(10):
        marks[seg].record()
        for _ in range(iters // 10):
            dst.copy_(src)
    marks[10].record()
    torch.cuda.synchronize()
    per_seg = 2.0 * nbytes * (iters // 10) / 1e9
    return per_seg / (marks[0].elapsed_time(marks[1]) * 1e-3), per_seg / (marks[9].elapsed_time(marks[10]) * 1e-3)


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons, power = [], [], set(), []
        for line in self.file.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.file.name)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


def chain_spec(name: str, sigma: float):
    return synth.config(name, sigma=sigma)


def verified_tokens(block_len) -> int:
    return int(block_len.clamp(min=0).sum().item())


def spread(ms):
    """mean / median / min of a list of per-step times in milliseconds, and the means of the first and the last tenth
    of the steps: a board that streams for tenths of a second may slow down under its power management, and the two
    tenths show whether this run met that."""
    out = {"mean": float(np.mean(ms)), "median": float(np.median(ms)), "min": float(np.min(ms))}
    n = len(ms) // 10
    if n >= 5:
        out["first_tenth_mean"] = float(np.mean(ms[:n]))
        out["last_tenth_mean"] = float(np.mean(ms[-n:]))
    return out


# ----------------------------------------------------------------------------------------- parity of the timed batch
def _cdf_distance(w, u, token):
    """Distance, in normalised CDF units, from u to `token`'s inverse-CDF interval under the weights w (inf for a zero-mass token)."""
    if token < 0 or token >= len(w) or not (w[token] > 0.0):
        return float("inf")
    c = np.cumsum(w)
    return float(max((c[token] - w[token]) / c[-1] - u, u - c[token] / c[-1], 0.0))


def _classify(ga, gn, oa, on, margin, sinfo, distance=None):
    """One (level, sequence) result against the oracle's: exact, a counted tie (a uniform within 1e-6 of its decision
    threshold; for a sample the other side's token must be the neighbouring positive-mass token or, where tokens are
    lighter than the band, one whose own interval lies within 1e-6 of the uniform), or a mismatch."""
    if ga == oa and gn == on:
        return "exact"
    if ga != oa:
        j = min(ga, oa)
        if 0 <= j < len(margin) and np.isfinite(margin[j]) and margin[j] <= TIE_BAND:
            return "tie_accept"
        return "mismatch"
    if sinfo[0] <= TIE_BAND and gn >= 0:
        if gn in (int(sinfo[2]), int(sinfo[3])) or (distance is not None and distance(gn) <= TIE_BAND):
            return "tie_sample"
    return "mismatch"


def parity_chain(gpu, ora, sample=None):
    """Counters over every (level, sequence) of a chain batch, bottom level first; after a tie the two sides walk
    different streams, so the levels above it are not compared.  `sample` (the oracle's inputs) lets a sampling tie
    among tokens lighter than the band be recognised from the float64 weights of the row pair."""
    from oracle import oracle as orc
    L, B = ora["accepted_len"].shape
    c = {"exact": 0, "tie_accept": 0, "tie_sample": 0, "mismatch": 0, "skipped_after_tie": 0, "compared": 0}

    def distance_at(l, b):
        if sample is None:
            return None

        def distance(token):
            a, m, T = int(ora["accepted_len"][l, b]), int(ora["block_len"][l, b]), sample["temperature"]
            P = orc.softmax_row(sample["models"][l][b, a], T)
            w = np.maximum(P - orc.softmax_row(sample["models"][l + 1][b, a], T), 0.0) if a < m else P
            return _cdf_distance(w if w.sum() > 0.0 else P, float(sample["uniforms"][l, b, -1]), int(token))
        return distance

    for b in range(B):
        for l in range(L - 1, -1, -1):
            ga, oa = int(gpu["accepted_len"][l, b]), int(ora["accepted_len"][l, b])
            kind = _classify(ga, int(gpu["out_tokens"][l, b, max(ga, 0)]), oa, int(ora["out_tokens"][l, b, max(oa, 0)]),
                             ora["accept_margin"][l, b], ora["sample_info"][l, b], distance_at(l, b))
            if kind == "exact" and not (gpu["block_len"][l, b] == ora["block_len"][l, b] and gpu["out_len"][l, b] == ora["out_len"][l, b]
                                        and (gpu["out_tokens"][l, b] == ora["out_tokens"][l, b]).all()):
                kind = "mismatch"
            c[kind] += 1
            c["compared"] += 1
            if kind != "exact":
                if kind != "mismatch":
                    c["skipped_after_tie"] += l
                break
    return c


def parity_level(gpu_a, gpu_next, ora):
    c = {"exact": 0, "tie_accept": 0, "tie_sample": 0, "mismatch": 0, "compared": 0}
    for b in range(len(ora["accepted_len"])):
        c[_classify(int(gpu_a[b]), int(gpu_next[b]), int(ora["accepted_len"][b]), int(ora["next_token"][b]),
                    ora["accept_margin"][b], ora["sample_info"][b])] += 1
        c["compared"] += 1
    return c


# ----------------------------------------------------------------------------------------- CPU oracle legs
def oracle_chain(sample, threads):
    from oracle import oracle as orc
    t0 = time.perf_counter()
    out = orc.verify_chain(sample["models"], sample["k"], sample["draft_tokens"], sample["uniforms"],
                           sample["temperature"], threads=threads)
    dt = time.perf_counter() - t0
    return int(out["block_len"].clip(min=0).sum()), dt, out


def cpu_baseline(data, spec, gpu_out, target_seconds=12.0):
    """The oracle, as it stands, on the resident batch: whole passes over it until about target_seconds of CPU
    work.  The first pass's outputs are compared with the GPU's outputs on the same batch (parity counters)."""
    from oracle import oracle as orc
    orc.build()
    cores = os.cpu_count() or 1
    sample = {"models": [m.cpu() for m in data["models"]], "k": data["k"], "draft_tokens": data["draft_tokens"].cpu(),
              "uniforms": data["uniforms"].cpu().contiguous(), "temperature": data["temperature"]}
    tok0, t0, out0 = oracle_chain(sample, cores)
    parity = parity_chain({k: v.cpu().numpy() for k, v in gpu_out.items() if k != "device_status"}, out0, sample)
    passes = int(min(200, max(1, round(target_seconds / max(t0, 1e-3)))))
    tok, t = tok0, t0
    for _ in range(passes - 1):
        a, b, _ = oracle_chain(sample, cores)
        tok += a
        t += b
    return {"value": tok / t, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{passes} passes over the {spec.B} sequences of the same batch, {tok} verified tokens in {t:.2f} s, "
                      f"{cores} threads (one sequence per thread at a time)"}, parity


def fused_oracle(d, n_seq, threads):
    from oracle import oracle as orc
    t0 = time.perf_counter()
    out = orc.verify_from_hidden(d["hidden_p"][:n_seq], d["W_p"], d["hidden_q"][:n_seq], d["W_q"], d["draft_tokens"][:n_seq].cpu(),
                                 d["uniforms"][:n_seq].cpu(), d["temperature"], threads=threads)
    dt = time.perf_counter() - t0
    return int(n_seq * d["draft_tokens"].shape[1]), dt, out


def fused_parity(got_a, got_next, logits_p_gpu, ora, d):
    """Strict counters (1e-6 band) plus, for the disagreements, how many the tensor core's fp32 accumulation
    explains: an accept uniform within 4 dl / T of min(1, P/Q), or a sampling uniform within 8 dl / (T S) of the GPU
    token's CDF interval under the oracle's logits (dl = measured max |logit difference|, S = residual mass)."""
    from scipy.special import softmax as sp_softmax
    c = parity_level(got_a, got_next, ora)
    dl = float((logits_p_gpu.double().cpu() - ora["logits_p"]).abs().max())
    T = d["temperature"]
    k = d["draft_tokens"].shape[1]
    u = d["uniforms"].cpu().numpy()
    band = max(4 * dl / T, TIE_BAND)
    explained = unexplained = 0
    for b in range(len(got_a)):
        ga, gn, oa, on = int(got_a[b]), int(got_next[b]), int(ora["accepted_len"][b]), int(ora["next_token"][b])
        if ga == oa and gn == on:
            continue
        if ga != oa:
            ok = ora["accept_margin"][b, min(ga, oa)] <= band
        else:
            P = sp_softmax(ora["logits_p"][b, oa].numpy() / T)
            w = np.maximum(P - sp_softmax(ora["logits_q"][b, oa].numpy() / T), 0.0) if oa < k else P
            cdf = np.cumsum(w)
            lo, hi = (cdf[gn] - w[gn]) / cdf[-1], cdf[gn] / cdf[-1]
            ok = w[gn] > 0 and max(lo - u[b, k], u[b, k] - hi, 0.0) <= 2 * band / w.sum()
        explained += bool(ok)
        unexplained += not ok
    c.update({"max_abs_logit_difference": dl, "explained_by_fp32_accumulation": explained, "unexplained": unexplained})
    return c


def run_reference(args, spec):
    """--impl reference: the CPU oracle, every step a whole pass over a bounded sample of the workload (several
    sequences per thread, so that a step does not wait on its slowest sequence alone)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle as orc
    orc.build()
    cores = os.cpu_count() or 1
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    if isinstance(spec, synth.FusedSpec):
        n_seq = min(spec.B, 4)
        d = synth.make_fused(spec, seed=args.seed, device=dev)
        d = {k: (v.cpu() if torch.is_tensor(v) else v) for k, v in d.items()}
        step = lambda: fused_oracle(d, n_seq, cores)[:2]
    else:
        n_seq = min(spec.B, 4 * cores)
        d = synth.make_chain(synth.scaled(spec, B=n_seq), seed=args.seed, device=dev)
        sample = {"models": [m.cpu() for m in d["models"]], "k": d["k"], "draft_tokens": d["draft_tokens"].cpu(),
                  "uniforms": d["uniforms"].cpu(), "temperature": d["temperature"]}
        step = lambda: oracle_chain(sample, cores)[:2]
    for _ in range(args.warmup):
        step()
    tokens, elapsed = 0, 0.0
    for _ in range(args.steps):
        tok, dt = step()
        tokens += tok
        elapsed += dt
    value = tokens / elapsed
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * elapsed / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(args, spec)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"the first {n_seq} of {spec.B} sequences of the recipe per step, {args.steps} steps, {cores} threads"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def workload_name(args, spec):
    if isinstance(spec, synth.FusedSpec):
        return (f"cfg4: fused LM-head verify, B={spec.B} per GPU, k={spec.k}, V={spec.V}, hidden bf16 [{spec.B},{spec.k + 1},{spec.d_p}] / "
                f"[{spec.B},{spec.rows_q},{spec.d_q}], LM-head weights bf16 [{spec.V},{spec.d_p}] / [{spec.V},{spec.d_q}], T={spec.temperature}")
    k_bottom_up = tuple(reversed(spec.k))
    extra = f", inter-level sigma {args.sigma}" if spec.name == "cfg5" else ""
    return (f"{spec.name}: {spec.n_models}-level chain, B={spec.B} per GPU, V={spec.V}, "
            f"{'bf16' if spec.dtype == torch.bfloat16 else 'fp32'} logits, k={k_bottom_up} bottom-up, "
            f"T={spec.temperature}{extra}")


def reduce_over_ranks(times_ms, work, device, world):
    """The multi-GPU bookkeeping: MAX over ranks of every time, SUM over ranks of every work count.

    Ranks verify disjoint batches and never exchange data on the path itself; this is the only
    collective of a run.  Returns two lists of floats (identical on every rank)."""
    import torch.distributed as dist
    t = torch.tensor(list(times_ms), device=device, dtype=torch.float64)
    w = torch.tensor(list(work), device=device, dtype=torch.float64)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(w, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], [float(x) for x in w.tolist()]


# ----------------------------------------------------------------------------------------- GPU arm
class Env:
    """Rank, device and process group of this process (one process per GPU)."""

    def __init__(self):
        from paper_2510_26527_b200 import binding, buildlib
        import torch.distributed as dist
        self.dist = dist
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        if not torch.cuda.is_available():
            raise RuntimeError("bench.py needs a CUDA device: libpolyspec has no CPU path")
        torch.cuda.set_device(self.local)
        self.dev = torch.device("cuda", self.local)
        if self.world > 1:
            dist.init_process_group("nccl", device_id=self.dev)
        if self.rank == 0:
            buildlib.build()
        if self.world > 1:
            dist.barrier()
        binding.load_library()
        self.binding = binding

    def barrier(self):
        if self.world > 1:
            self.dist.barrier()
        torch.cuda.synchronize()

    def close(self):
        if self.world > 1:
            self.dist.destroy_process_group()


def timed_region(env, calls, parts_of, steps, sample_clocks):
    """K steps between two events, step i on calls[i % len(calls)], with an event after every part of a step
    (parts_of(call) -> list of (name, function)).  Returns total ms, per-step ms, per-part mean ms, clocks."""
    names = [n for n, _ in parts_of(calls[0])]
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(len(names) + 1)] for _ in range(steps)]
    fns = [[f for _, f in parts_of(c)] for c in calls]
    sampler = ClockSampler(env.local)
    env.barrier()
    if env.rank == 0 and sample_clocks:
        sampler.start()
        time.sleep(0.3)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    env.barrier()
    start.record()
    for i in range(steps):
        f = fns[i % len(fns)]
        ev[i][0].record()
        for j, fn in enumerate(f):
            fn()
            ev[i][j + 1].record()
    stop.record()
    env.barrier()
    total = start.elapsed_time(stop)
    clocks = sampler.stop() if (env.rank == 0 and sample_clocks) else None
    per_step = [e[0].elapsed_time(e[-1]) for e in ev]
    per_part = {n: sum(e[j].elapsed_time(e[j + 1]) for e in ev) / steps for j, n in enumerate(names)}
    return total, per_step, per_part, clocks


def chain_parts(call):
    return [("row_stats", call.row_stats), ("walk", call.walk)]


def measure_chain(env, args, spec, steps, warmup, headline):
    """One logits-path workload on this rank's own batch.  Returns the record (rank 0) of the JSON line."""
    binding, dev, rank, world = env.binding, env.dev, env.rank, env.world
    # sequences are independent: each rank verifies its own batch, no data-path collective
    data = synth.make_chain(spec, seed=args.seed, device=dev, batch_offset=rank * spec.B)
    call = binding.ChainCall(data["models"], data["k"], data["draft_tokens"], data["uniforms"], data["temperature"])
    logits_bytes = spec.logits_bytes()
    fits_l2 = logits_bytes <= 2 * 126e6

    for _ in range(max(warmup, 3)):
        call.launch()
    torch.cuda.synchronize()
    tokens_per_step = verified_tokens(call.out["block_len"])
    emitted_per_step = int(call.out["out_len"][0].sum().item())
    assert int(call.device_status.item()) == 0

    # ---- device-timed region: K steps, each exactly polyspec_verify_chain (its two halves, with an event between
    # them so that the dominant kernel's share is measured live)
    elapsed_ms, per_step, per_part, clocks = timed_region(env, [call], chain_parts, steps, True)
    stats_ms, walk_ms = per_part["row_stats"], per_part["walk"]
    # the same steps as single C-ABI calls, no event inside a step
    whole_ms, whole_steps, _, _ = timed_region(env, [call], lambda c: [("call", c.launch)], steps, False)

    # ---- inputs that fit in L2 (the batch-1 workloads): also as a replayed CUDA graph of ten calls, which is how a
    # decode loop would issue a step this short, and which takes the host's launch cost out of the figure
    graph = None
    if fits_l2 and world == 1:
        side = torch.cuda.Stream(device=dev)
        gcall = binding.ChainCall(data["models"], data["k"], data["draft_tokens"], data["uniforms"], data["temperature"],
                                  stream=side.cuda_stream)
        with torch.cuda.stream(side):
            gcall.launch()
            side.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for _ in range(10):
                    gcall.launch()
            for _ in range(5):
                g.replay()
            side.synchronize()
            reps = max(20, steps // 10)
            marks = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
            marks[0].record(side)
            for i in range(reps):
                g.replay()
                marks[i + 1].record(side)
            side.synchronize()
        same_graph = all(torch.equal(gcall.out[n], call.out[n]) for n in ("accepted_len", "block_len", "out_tokens", "out_len"))
        graph = {"calls_per_graph": 10, "replays": reps, "matches_plain_calls": bool(same_graph),
                 "us_per_call": spread([100.0 * marks[i].elapsed_time(marks[i + 1]) for i in range(reps)])}

    # ---- inputs that fit in L2: also L2-cold, rotating through >= 256 MB of distinct instances of the workload
    cold = None
    if fits_l2 and world == 1:
        n_inst = int(256e6 // logits_bytes) + 1
        many = synth.make_chain(synth.scaled(spec, B=spec.B * n_inst), seed=args.seed + 1, device=dev)
        inst = []
        for i in range(n_inst):
            s = slice(i * spec.B, (i + 1) * spec.B)
            inst.append(binding.ChainCall([m[s] for m in many["models"]], many["k"], many["draft_tokens"][s].contiguous(),
                                          many["uniforms"][:, s].contiguous(), many["temperature"]))
        for c in inst:
            c.launch()
        torch.cuda.synchronize()
        cold_ms, cold_steps, _, _ = timed_region(env, inst, lambda c: [("call", c.launch)], max(steps, n_inst), False)
        cold = {"us_per_call": spread([1e3 * x for x in cold_steps]), "instances": n_inst,
                "distinct_bytes": n_inst * logits_bytes, "steps": max(steps, n_inst)}
        del inst, many

    # ---- end to end (headline only): the host-buffer entry point, H2D of every input and D2H of every output inside the region
    e2e = None
    if headline:
        e2e_steps = max(1, min(steps, args.e2e_steps))
        host_models = [m.cpu().pin_memory() for m in data["models"]]
        host_tok, host_u = data["draft_tokens"].cpu().pin_memory(), data["uniforms"].cpu().pin_memory()
        rows = [int(m.shape[1]) for m in host_models]
        ws_bytes = binding.polyspec_verify_chain_host_workspace(data["k"], rows, spec.B, spec.V, call.dt)
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        host_out = binding.chain_outputs(spec.n_models - 1, spec.B, spec.kmax, "cpu", pin=True)
        h2d = sum(m.numel() * m.element_size() for m in host_models) + host_tok.numel() * 4 + host_u.numel() * 4
        d2h = sum(v.numel() * 4 for v in host_out.values()) + 4
        binding.polyspec_verify_chain_host(host_models, data["k"], host_tok, host_u, data["temperature"], ws, out=host_out)
        env.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e2e_steps):
            binding.polyspec_verify_chain_host(host_models, data["k"], host_tok, host_u, data["temperature"], ws, out=host_out)
        e1.record()
        env.barrier()
        e2e_ms = e0.elapsed_time(e1)
        same = all(bool((host_out[k].to(dev) == call.out[k]).all()) for k in ("accepted_len", "block_len", "out_tokens", "out_len"))
        del ws, host_models
    else:
        e2e_ms, e2e_steps, h2d, d2h, same = 0.0, 1, 0, 0, None

    # ---- reduce over ranks: max time, summed work
    (elapsed_ms, whole_ms, e2e_ms, stats_ms, walk_ms), (tokens_all, emitted_all) = reduce_over_ranks(
        [elapsed_ms, whole_ms, e2e_ms, stats_ms, walk_ms], [tokens_per_step, emitted_per_step], dev, world)

    base = parity = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:      # the CPU baseline and the parity check are one-GPU-run extras
        base, parity = cpu_baseline(data, spec, call.out, target_seconds=args.cpu_seconds if headline else 2.0)

    if rank != 0:
        return None
    peaks = read_peaks()
    ms_per_step = elapsed_ms / steps
    achieved = logits_bytes / (stats_ms * 1e-3) / 1e9
    traffic = None if STATS_TRAFFIC_PER_LOGIT_BYTE is None else STATS_TRAFFIC_PER_LOGIT_BYTE * logits_bytes
    rec = {
        "metric": METRIC, "value": tokens_all * steps / (elapsed_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": max(warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name(args, spec), "seed": args.seed,
                   "l2": ("inputs fit in L2: L2-warm timing (the same instance every step); the L2-cold figure is under l2_cold" if fits_l2 else
                          f"inputs {logits_bytes / 1e9:.3f} GB per step, larger than the 126 MB L2; no flush needed"),
                   "parallelism": f"{world} independent replicas, batch sharded, no collective"},
        "gpu_launches": 2 * steps,
        "step_ms": spread(per_step),
        "single_call_step_ms": dict(spread(whole_steps), total_over_steps=whole_ms / steps),
        "emitted_tokens_per_s": emitted_all * steps / (elapsed_ms * 1e-3),
        "whole_step_gbs": logits_bytes * world / (ms_per_step * 1e-3) / 1e9,
        "whole_step_frac_of_hbm_peak": logits_bytes / (ms_per_step * 1e-3) / 1e9 / peaks["hbm_gbs"],
        "kernel_ms": {"row_stats": stats_ms, "walk": walk_ms},
        "roofline": {"bound": "hbm", "kernel": "stats_kernel (row statistics, every logit once)",
                     "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                     "traffic": traffic, "peak_source": f"of {peaks['source']}",
                     "frac_of_nominal_8TBs": achieved / 8000.0},
        "clocks": clocks,
    }
    if cold is not None:
        rec["l2_cold"] = cold
    if graph is not None:
        rec["cuda_graph"] = graph
    if headline:
        live_copy = copy_probe_gbs(dev)
        copy_first, copy_last = copy_probe_sustained_gbs(dev)
        rec["roofline"].update({"this_gpu_copy_gbs": live_copy, "frac_of_this_gpu_copy": achieved / live_copy,
                                "this_gpu_copy_sustained_gbs": {"first_tenth": copy_first, "last_tenth": copy_last},
                                "frac_of_this_gpu_sustained_copy": achieved / copy_last})
        rec["e2e"] = {"value": tokens_all * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                      "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps,
                      "matches_device_path": same}
    if base is not None:
        rec["cpu_baseline"] = base
        rec["parity"] = parity
    return rec


def measure_fused(env, args, spec, steps, warmup, headline):
    """cfg4: hidden states -> LM-head projections on the tensor cores -> verification, one C-ABI call per step."""
    binding, dev, rank, world = env.binding, env.dev, env.rank, env.world
    d = synth.make_fused(spec, seed=args.seed + 7919 * rank, device=dev)
    call = binding.FusedCall(d["hidden_p"], d["W_p"], d["hidden_q"], d["W_q"], d["draft_tokens"], d["uniforms"], d["temperature"])
    for _ in range(max(warmup, 3)):
        call.launch()
    torch.cuda.synchronize()
    assert int(call.device_status.item()) == 0
    tokens_per_step = spec.B * spec.k
    emitted_per_step = int((call.out["accepted_len"] + 1).sum().item())

    elapsed_ms, per_step, per_part, clocks = timed_region(
        env, [call], lambda c: [("lm_head_project_with_row_stats", c.project), ("walk", c.verify)], steps, True)
    gemm_ms, verify_ms = per_part["lm_head_project_with_row_stats"], per_part["walk"]
    whole_ms, whole_steps, _, _ = timed_region(env, [call], lambda c: [("call", c.launch)], steps, False)

    # end to end: this step's hidden states, draft tokens and uniforms come from pinned host memory, the
    # outputs go back to pinned host memory; the LM-head weights are model parameters and stay resident
    e2e_steps = max(1, min(steps, args.e2e_steps))
    host_in = [t.cpu().pin_memory() for t in (d["hidden_p"], d["hidden_q"], d["draft_tokens"], d["uniforms"])]
    dev_in = [d["hidden_p"], d["hidden_q"], d["draft_tokens"], d["uniforms"]]
    host_out = [torch.empty(spec.B, dtype=torch.int32).pin_memory() for _ in range(2)]
    h2d = sum(t.numel() * t.element_size() for t in host_in)
    d2h = 2 * spec.B * 4

    def e2e_step():
        for h, g in zip(host_in, dev_in):
            g.copy_(h, non_blocking=True)
        call.launch()
        host_out[0].copy_(call.out["accepted_len"], non_blocking=True)
        host_out[1].copy_(call.out["next_token"], non_blocking=True)
    e2e_step()
    env.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e1.record()
    env.barrier()
    e2e_ms = e0.elapsed_time(e1)

    (elapsed_ms, whole_ms, e2e_ms, gemm_ms, verify_ms), (tokens_all, emitted_all) = reduce_over_ranks(
        [elapsed_ms, whole_ms, e2e_ms, gemm_ms, verify_ms], [tokens_per_step, emitted_per_step], dev, world)

    base = parity = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import oracle as orc
        orc.build()
        cores = os.cpu_count() or 1
        dc = {k: (v.cpu() if torch.is_tensor(v) else v) for k, v in d.items()}
        tok, t, ora = fused_oracle(dc, spec.B, cores)        # the whole timed batch: parity and the baseline in one pass
        lp, _ = binding.polyspec_lm_head(d["hidden_p"], d["W_p"])
        torch.cuda.synchronize()
        parity = fused_parity(call.out["accepted_len"].cpu().numpy(), call.out["next_token"].cpu().numpy(), lp, ora, dc)
        base = {"value": tok / t, "unit": UNIT, "cores": cores, "kind": "oracle",
                "sample": f"all {spec.B} sequences of the same batch, once (float64 matmul of the LM head on the host, then the "
                          f"verification rule), {tok} verified tokens in {t:.2f} s, {cores} threads"}

    if rank != 0:
        return None
    peaks = read_peaks()
    ms_per_step = elapsed_ms / steps
    flops = spec.flops()
    achieved = flops / (gemm_ms * 1e-3) / 1e12
    call_ms = whole_ms / steps
    rec = {
        "metric": METRIC, "value": tokens_all * steps / (elapsed_ms * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": steps, "warmup": max(warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload_name(args, spec), "seed": args.seed,
                   "l2": f"inputs {(spec.weight_bytes() + 2 * spec.B * (spec.k + 1) * (spec.d_p + spec.d_q)) / 1e9:.3f} GB per step, "
                         "larger than the 126 MB L2; no flush needed",
                   "parallelism": f"{world} independent replicas, batch sharded, no collective"},
        "gpu_launches": 2 * steps,
        "step_ms": spread(per_step),
        "single_call_step_ms": dict(spread(whole_steps), total_over_steps=call_ms),
        "emitted_tokens_per_s": emitted_all * steps / (elapsed_ms * 1e-3),
        "whole_step_tflops": flops * world / (ms_per_step * 1e-3) / 1e12,
        "whole_step_frac_of_tensor_peak": flops / (ms_per_step * 1e-3) / 1e12 / peaks["bf16_tflops"],
        "whole_step_frac_of_sustained_tensor_peak": flops / (ms_per_step * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
        "single_call_frac_of_tensor_peak": flops / (call_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
        "kernel_ms": {"lm_head_project_with_row_stats": gemm_ms, "walk": verify_ms},
        "roofline": {"bound": "tensor", "kernel": "lmhead_kernel (both LM-head projections, tcgen05 cta_group::2)",
                     "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                     "frac_of_sustained_peak": achieved / peaks["bf16_tflops_sustained"],
                     "traffic": LMHEAD_TRAFFIC_BYTES, "peak_source": f"of {peaks['source']} (burst)",
                     "weight_stream_gbs": spec.weight_bytes() / (gemm_ms * 1e-3) / 1e9,
                     "weight_stream_frac_of_hbm_peak": spec.weight_bytes() / (gemm_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
        "e2e": {"value": tokens_all * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps,
                "note": "hidden states, tokens and uniforms copied per step; LM-head weights resident"},
        "clocks": clocks,
    }
    if base is not None:
        rec["cpu_baseline"] = base
        rec["parity"] = parity
    return rec


def run_gpu(args, spec):
    env = Env()
    fused = isinstance(spec, synth.FusedSpec)
    line = (measure_fused if fused else measure_chain)(env, args, spec, args.steps, args.warmup, True)
    # a default run (one GPU, the headline workload) also measures the other four configurations, briefly
    if env.world == 1 and args.workload == "cfg5" and args.batch == 0 and not args.no_workloads:
        others = {}
        for name in ("cfg1", "cfg2", "cfg3", "cfg4"):
            torch.cuda.empty_cache()
            sp = synth.FusedSpec() if name == "cfg4" else chain_spec(name, args.sigma)
            rec = (measure_fused if name == "cfg4" else measure_chain)(env, args, sp, args.workload_steps, 5, False)
            for drop in ("metric", "unit", "n_gpus", "higher_is_better", "scaling", "vs_baseline", "data"):
                rec.pop(drop, None)
            rec["us_per_step"] = 1e3 * rec["ms_per_step"]
            others[name] = rec
        line["workloads"] = others
    if env.rank == 0:
        print(json.dumps(line))
    env.close()


def run_gpu_greedy(args, spec):
    """--rule greedy: the chain under greedy matching (one arg-max pass over the verifiers' logits + a small walk)."""
    from paper_2510_26527_b200 import binding, buildlib
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: libpolyspec has no CPU path")
    if int(os.environ.get("WORLD_SIZE", "1")) != 1:
        raise RuntimeError("--rule greedy is a single-GPU measurement")
    dev = torch.device("cuda", 0)
    buildlib.build()
    binding.load_library()
    data = synth.make_chain(spec, seed=args.seed, device=dev)
    kb = data["k"][-1]
    g = torch.Generator(device=dev).manual_seed(args.seed + 1)
    top = data["models"][-2][:, :kb].float().argmax(-1)
    flip = torch.rand(top.shape, generator=g, device=dev) < 0.1
    draft = torch.where(flip, torch.randint(0, spec.V, top.shape, generator=g, device=dev), top).to(torch.int32).contiguous()
    verifiers = data["models"][:-1]
    rows = [int(m.shape[1]) for m in verifiers] + [kb]
    ws = torch.empty(max(256, binding.polyspec_verify_chain_greedy_workspace(data["k"], rows, spec.B, spec.V, binding._dt(verifiers[0]))),
                     dtype=torch.uint8, device=dev)
    out = binding.chain_outputs(spec.n_models - 1, spec.B, spec.kmax, dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    call = lambda: binding.polyspec_verify_chain_greedy(data["models"], data["k"], draft, workspace=ws, out=out, device_status=status)
    for _ in range(max(args.warmup, 3)):
        call()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(args.steps):
        call()
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / args.steps
    peaks = read_peaks()
    elem = 4 if spec.dtype == torch.float32 else 2
    vbytes = sum(int(m.shape[1]) for m in verifiers) * spec.B * spec.V * elem
    tokens = verified_tokens(out["block_len"])
    achieved = vbytes / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": METRIC, "value": tokens / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name(args, spec) + ", greedy matching (verifier rows only)", "seed": args.seed},
        "gpu_launches": 2 * args.steps, "mean_accepted_len_top_level": float(out["accepted_len"][0].float().mean()),
        "roofline": {"bound": "hbm", "kernel": "stats_kernel in arg-max mode + greedy walk (whole call)", "achieved": achieved,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "traffic": None,
                     "peak_source": f"of {peaks['source']}"},
        "clocks": clocks}))


# ----------------------------------------------------------------------------------------- launcher
def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_ranks(n: int, argv) -> int:
    """`--gpus N` without a launcher: start N ranks of this script (one process per GPU) on this node and
    return their exit status.  The ranks are independent replicas; they meet only to combine times and counts."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def launch_check():
    """What a multi-rank run adds on the host, without any kernel: rendezvous, the MAX / SUM reduction and rank 0's
    single line.  Runs on `gloo` when there is no GPU (the CPU test of the launcher uses it)."""
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    use_cuda = torch.cuda.is_available()
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0"))) if use_cuda else torch.device("cpu")
    if world > 1:
        dist.init_process_group("nccl" if use_cuda else "gloo")
    (t_max,), (work,) = reduce_over_ranks([10.0 + rank], [100 * (rank + 1)], dev, world)
    if rank == 0:
        print(json.dumps({"launch_check": True, "n_gpus": world, "max_ms": t_max, "summed_work": work}))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main(argv=None):
    argv = sys.argv[1:] if argv is None else list(argv)
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="polyspec", choices=["polyspec", "reference"])
    ap.add_argument("--workload", default="cfg5", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--sigma", type=float, default=1.0, help="inter-level noise of cfg5")
    ap.add_argument("--rule", default="sampling", choices=["sampling", "greedy"],
                    help="verification rule; greedy matching is timed on the logits-path workloads only")
    ap.add_argument("--batch", type=int, default=0,
                    help="override the batch of a logits-path workload (e.g. 512 stacked instances of the batch-1 configs)")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-workloads", action="store_true", help="headline workload only")
    ap.add_argument("--workload-steps", type=int, default=1000, help="steps of each of the other configurations in a default run")
    ap.add_argument("--launch-check", action="store_true", help="rendezvous and reduction only (no kernels)")
    args = ap.parse_args(argv)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        sys.exit(launch_ranks(args.gpus, argv))
    if args.launch_check:
        return launch_check()
    spec = synth.FusedSpec() if args.workload == "cfg4" else chain_spec(args.workload, args.sigma)
    if args.batch > 0 and args.workload != "cfg4":
        spec = synth.scaled(spec, B=args.batch)
    if args.impl == "reference":
        run_reference(args, spec)
    elif args.rule == "greedy" and args.workload != "cfg4":
        run_gpu_greedy(args, spec)
    else:
        run_gpu(args, spec)


if __name__ == "__main__":
    main()
