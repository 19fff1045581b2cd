#!/usr/bin/env python
"""Benchmark of the chained verification step (libpolyspec) on synthetic logits.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5|cfg3|cfg2|cfg1|cfg4] [--impl reference]

`--workload cfg4` is the fused path (hidden states -> LM-head projections on the tensor cores -> verification); its
roofline object is the tensor one.

One step = one pass of the whole hot path (row statistics over every logits row of every model,
then accept tests / first rejection / replacement-or-bonus sampling / hand-off for every level)
over one batch that is already resident in HBM.  The default workload is the largest logits-path
configuration, the four-level chain (B=256 per GPU, V=152064, bf16, k=(10,6,4) bottom-up, 2.57 GB of
logits per call -- larger than L2, so nothing is served from cache between steps).

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle as it stands on the host
cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2510_26527_b200 import synth  # noqa: E402

METRIC = "verified_draft_tokens_per_s"
UNIT = "tokens/s"

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the row-statistics kernel, from the ncu
# capture summarised under profiles/ (bytes per logits byte processed, measured on a smaller case of
# the same kernel and scaled by the bytes one launch processes).  None until a capture exists.
STATS_TRAFFIC_PER_LOGIT_BYTE = 1.0130     # profiles/stats_kernel_bf16_cfg3_ncu_full.md: (328.350 + 4.250) MB moved for 328.340 MB of logits
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


# ----------------------------------------------------------------------------------------- CPU oracle legs
def oracle_sample(spec, seed, n_seq, device):
    """The first n_seq sequences of the recipe (same V, rows, dtype), as CPU tensors."""
    d = synth.make_chain(synth.scaled(spec, B=n_seq), seed=seed, device=device)
    return {"models": [m.cpu() for m in d["models"]], "k": d["k"], "draft_tokens": d["draft_tokens"].cpu(),
            "uniforms": d["uniforms"].cpu(), "temperature": d["temperature"]}


def oracle_time(sample, threads):
    from oracle import oracle as orc
    t0 = time.perf_counter()
    out = orc.verify_chain(sample["models"], sample["k"], sample["draft_tokens"], sample["uniforms"],
                           sample["temperature"], threads=threads)
    dt = time.perf_counter() - t0
    return int(out["block_len"].clip(min=0).sum()), dt


def cpu_baseline(data, spec, target_seconds=12.0):
    """The oracle, as it stands, on the resident batch: whole passes over it until about target_seconds of CPU work."""
    from oracle import oracle as orc
    orc.build()
    cores = os.cpu_count() or 1
    sample = {"models": [m.cpu() for m in data["models"]], "k": data["k"], "draft_tokens": data["draft_tokens"].cpu(),
              "uniforms": data["uniforms"].cpu().contiguous(), "temperature": data["temperature"]}
    tok0, t0 = oracle_time(sample, cores)
    passes = int(min(200, max(1, round(target_seconds / max(t0, 1e-3)))))
    tok, t = 0, 0.0
    for _ in range(passes):
        a, b = oracle_time(sample, cores)
        tok += a
        t += b
    return {"value": tok / t, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{passes} passes over the {spec.B} sequences of the same batch, {tok} verified tokens in {t:.2f} s, "
                      f"{cores} threads (one sequence per thread)"}


def fused_oracle_time(d, n_seq, threads):
    from oracle import oracle as orc
    t0 = time.perf_counter()
    out = orc.verify_from_hidden(d["hidden_p"][:n_seq], d["W_p"], d["hidden_q"][:n_seq], d["W_q"], d["draft_tokens"][:n_seq].cpu(),
                                 d["uniforms"][:n_seq].cpu(), d["temperature"], threads=threads)
    dt = time.perf_counter() - t0
    return int(n_seq * d["draft_tokens"].shape[1]), dt, out


def fused_cpu_baseline(d, spec, target_seconds=12.0):
    """The oracle's float64 projection + verification on the first sequences of the batch."""
    from oracle import oracle as orc
    orc.build()
    cores = os.cpu_count() or 1
    n0 = min(spec.B, 2)
    tok0, t0, _ = fused_oracle_time(d, n0, cores)
    n = int(min(spec.B, max(n0, n0 * target_seconds / max(t0, 1e-3))))
    tok, t, _ = fused_oracle_time(d, n, cores)
    return {"value": tok / t, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {n} of {spec.B} sequences of the same batch (float64 matmul of the LM head on the host, then the "
                      f"verification rule), {tok} verified tokens in {t:.2f} s, {cores} threads"}


def run_reference(args, spec):
    """--impl reference: the CPU oracle on a bounded sample per step."""
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
        step = lambda: fused_oracle_time(d, n_seq, cores)[:2]
    else:
        n_seq = min(spec.B, cores)          # one sequence per thread: a step of some tens of milliseconds
        sample = oracle_sample(spec, seed=args.seed, n_seq=n_seq, device=dev)
        step = lambda: oracle_time(sample, cores)
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
        "config": {"workload": workload_name(args, spec), "sample": f"{n_seq} sequences per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{n_seq} of {spec.B} sequences of the recipe per step, {args.steps} steps"},
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
def run_gpu(args, spec):
    from paper_2510_26527_b200 import binding, buildlib
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: libpolyspec has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        buildlib.build()
    if world > 1:
        dist.barrier()
    binding.load_library()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # sequences are independent: each rank verifies its own batch, no data-path collective
    data = synth.make_chain(spec, seed=args.seed, device=dev, batch_offset=rank * spec.B)
    call = binding.ChainCall(data["models"], data["k"], data["draft_tokens"], data["uniforms"], data["temperature"])
    logits_bytes = spec.logits_bytes()

    for _ in range(max(args.warmup, 3)):
        call.launch()
    torch.cuda.synchronize()
    tokens_per_step = verified_tokens(call.out["block_len"])
    emitted_per_step = int(call.out["out_len"][0].sum().item())
    assert int(call.device_status.item()) == 0

    # ---- device-timed region: K steps, each = row_stats + walk (exactly polyspec_verify_chain), with an
    # event between the two halves so the dominant kernel's share is measured live
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local)
    barrier()
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    start.record()
    for i in range(args.steps):
        ev[i][0].record()
        call.row_stats()
        ev[i][1].record()
        call.walk()
        ev[i][2].record()
    stop.record()
    barrier()
    elapsed_ms = start.elapsed_time(stop)
    clocks = sampler.stop() if rank == 0 else None
    stats_ms = sum(e[0].elapsed_time(e[1]) for e in ev) / args.steps
    walk_ms = sum(e[1].elapsed_time(e[2]) for e in ev) / args.steps

    # ---- end to end: the host-buffer entry point, H2D of every input and D2H of every output inside the region
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    host_models = [m.cpu().pin_memory() for m in data["models"]]
    host_tok, host_u = data["draft_tokens"].cpu().pin_memory(), data["uniforms"].cpu().pin_memory()
    rows = [int(m.shape[1]) for m in host_models]
    ws_bytes = binding.polyspec_verify_chain_host_workspace(data["k"], rows, spec.B, spec.V, call.dt)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    host_out = binding.chain_outputs(spec.n_models - 1, spec.B, spec.kmax, "cpu", pin=True)
    h2d = sum(m.numel() * m.element_size() for m in host_models) + host_tok.numel() * 4 + host_u.numel() * 4
    d2h = sum(v.numel() * 4 for v in host_out.values()) + 4
    binding.polyspec_verify_chain_host(host_models, data["k"], host_tok, host_u, data["temperature"], ws, out=host_out)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        binding.polyspec_verify_chain_host(host_models, data["k"], host_tok, host_u, data["temperature"], ws, out=host_out)
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    same = all(bool((host_out[k].to(dev) == call.out[k]).all()) for k in ("accepted_len", "block_len", "out_tokens", "out_len"))
    del ws, host_models

    # ---- reduce over ranks: max time, summed work
    (elapsed_ms, e2e_ms, stats_ms, walk_ms), (tokens_all, emitted_all) = reduce_over_ranks(
        [elapsed_ms, e2e_ms, stats_ms, walk_ms], [tokens_per_step, emitted_per_step], dev, world)

    base = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:      # the CPU baseline is a one-GPU-run extra
        base = cpu_baseline(data, spec, target_seconds=args.cpu_seconds)

    if rank == 0:
        peaks = read_peaks()
        ms_per_step = elapsed_ms / args.steps
        value = tokens_all * args.steps / (elapsed_ms * 1e-3)
        achieved = logits_bytes / (stats_ms * 1e-3) / 1e9
        live_copy = copy_probe_gbs(dev)
        traffic = None if STATS_TRAFFIC_PER_LOGIT_BYTE is None else STATS_TRAFFIC_PER_LOGIT_BYTE * logits_bytes
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_name(args, spec), "seed": args.seed,
                       "l2": f"inputs {logits_bytes / 1e9:.3f} GB per step, larger than the 126 MB L2; no flush needed"
                             if logits_bytes > 2 * 126e6 else "inputs fit in L2: L2-warm timing",
                       "parallelism": f"{world} independent replicas, batch sharded, no collective"},
            "gpu_launches": 2 * args.steps,
            "emitted_tokens_per_s": emitted_all * args.steps / (elapsed_ms * 1e-3),
            "whole_step_gbs": logits_bytes * world / (ms_per_step * 1e-3) / 1e9,
            "whole_step_frac_of_hbm_peak": logits_bytes / (ms_per_step * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "kernel_ms": {"row_stats": stats_ms, "walk": walk_ms},
            "roofline": {"bound": "hbm", "kernel": "stats_kernel (row statistics, every logit once)",
                         "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                         "traffic": traffic, "peak_source": f"of {peaks['source']}",
                         "frac_of_nominal_8TBs": achieved / 8000.0,
                         "this_gpu_copy_gbs": live_copy, "frac_of_this_gpu_copy": achieved / live_copy},
            "e2e": {"value": tokens_all * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps,
                    "matches_device_path": same},
            "clocks": clocks,
        }
        if base is not None:
            line["cpu_baseline"] = base
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_gpu_fused(args, spec):
    """cfg4: hidden states -> LM-head projections on the tensor cores -> verification, one C-ABI call per step."""
    from paper_2510_26527_b200 import binding, buildlib
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: libpolyspec has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        buildlib.build()
    if world > 1:
        dist.barrier()
    binding.load_library()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    d = synth.make_fused(spec, seed=args.seed + 7919 * rank, device=dev)
    call = binding.FusedCall(d["hidden_p"], d["W_p"], d["hidden_q"], d["W_q"], d["draft_tokens"], d["uniforms"], d["temperature"])
    for _ in range(max(args.warmup, 3)):
        call.launch()
    torch.cuda.synchronize()
    assert int(call.device_status.item()) == 0
    tokens_per_step = spec.B * spec.k
    emitted_per_step = int((call.out["accepted_len"] + 1).sum().item())

    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local)
    barrier()
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    start.record()
    for i in range(args.steps):
        ev[i][0].record()
        call.project()
        ev[i][1].record()
        call.verify()
        ev[i][2].record()
    stop.record()
    barrier()
    elapsed_ms = start.elapsed_time(stop)
    clocks = sampler.stop() if rank == 0 else None
    gemm_ms = sum(e[0].elapsed_time(e[1]) for e in ev) / args.steps
    verify_ms = sum(e[1].elapsed_time(e[2]) for e in ev) / args.steps

    # end to end: this step's hidden states, draft tokens and uniforms come from pinned host memory, the
    # outputs go back to pinned host memory; the LM-head weights are model parameters and stay resident
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
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
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)

    (elapsed_ms, e2e_ms, gemm_ms, verify_ms), (tokens_all, emitted_all) = reduce_over_ranks(
        [elapsed_ms, e2e_ms, gemm_ms, verify_ms], [tokens_per_step, emitted_per_step], dev, world)

    base = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:      # the CPU baseline is a one-GPU-run extra
        base = fused_cpu_baseline({k: (v.cpu() if torch.is_tensor(v) else v) for k, v in d.items()}, spec, target_seconds=args.cpu_seconds)

    if rank == 0:
        peaks = read_peaks()
        ms_per_step = elapsed_ms / args.steps
        flops = spec.flops()
        achieved = flops / (gemm_ms * 1e-3) / 1e12
        line = {
            "metric": METRIC, "value": tokens_all * args.steps / (elapsed_ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(args, spec), "seed": args.seed,
                       "l2": f"inputs {(spec.weight_bytes() + 2 * spec.B * (spec.k + 1) * (spec.d_p + spec.d_q)) / 1e9:.3f} GB per step, "
                             "larger than the 126 MB L2; no flush needed",
                       "parallelism": f"{world} independent replicas, batch sharded, no collective"},
            "gpu_launches": 2 * args.steps,
            "emitted_tokens_per_s": emitted_all * args.steps / (elapsed_ms * 1e-3),
            "whole_step_tflops": flops * world / (ms_per_step * 1e-3) / 1e12,
            "whole_step_frac_of_tensor_peak": flops / (ms_per_step * 1e-3) / 1e12 / peaks["bf16_tflops"],
            "kernel_ms": {"lm_head_project_with_row_stats": gemm_ms, "walk": verify_ms},
            "roofline": {"bound": "tensor", "kernel": "lmhead_kernel (both LM-head projections, tcgen05 cta_group::2)",
                         "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                         "traffic": LMHEAD_TRAFFIC_BYTES, "peak_source": f"of {peaks['source']} (burst)",
                         "weight_stream_gbs": spec.weight_bytes() / (gemm_ms * 1e-3) / 1e9,
                         "weight_stream_frac_of_hbm_peak": spec.weight_bytes() / (gemm_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
            "e2e": {"value": tokens_all * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps,
                    "note": "hidden states, tokens and uniforms copied per step; LM-head weights resident"},
            "clocks": clocks,
        }
        if base is not None:
            line["cpu_baseline"] = base
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


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


def main():
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
    args = ap.parse_args()
    spec = synth.FusedSpec() if args.workload == "cfg4" else chain_spec(args.workload, args.sigma)
    if args.batch > 0 and args.workload != "cfg4":
        spec = synth.scaled(spec, B=args.batch)
    if args.impl == "reference":
        run_reference(args, spec)
    elif args.rule == "greedy" and args.workload != "cfg4":
        run_gpu_greedy(args, spec)
    elif args.workload == "cfg4":
        run_gpu_fused(args, spec)
    else:
        run_gpu(args, spec)


if __name__ == "__main__":
    main()
