#!/usr/bin/env python
"""Benchmark of the GDN backward (gdn_bwd through the C ABI) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1] [--impl ours|reference]

One step = one full gdn_bwd call (recompute stages + reverse-state scan + intra-chunk gradients) over
one synthetic batch of the chosen configuration.  Prints ONE JSON line (rank 0).  With N > 1 (launched
by torch.distributed.run) every rank processes its own independent batch of the same shape: chains are
independent, there is no data-path collective, scaling is weak.

`--impl reference` times the CPU fp64 oracle as it stands on the host cores, on a bounded sample of the
same workload (it is a deliberately slow program: a baseline, not a target).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "gdn_bwd_tokens_per_sec"
UNIT = "tokens/s"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=1, help="benchmark configuration index (0..4); 1 is the headline")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (used when profiling)")
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="target CPU time of the oracle sample")
    return ap.parse_args()


def workload_config(wl):
    return {"workload": wl.name, "dtype_io": wl.dtype, "B": wl.B, "T": wl.T, "H": wl.H, "d_k": wl.d_k, "d_v": wl.d_v,
            "chunk": wl.chunk, "n_sequences": wl.N, "tokens": wl.tokens, "delta_rule": wl.delta_rule,
            "varlen": wl.varlen, "seed": wl.seed,
            "l2": "inputs+outputs+workspace per step exceed the 126 MB L2; no explicit flush"}


def time_oracle_sample(wl, target_seconds):
    """Times the oracle on the first h heads of the workload, h chosen from a one-head calibration run."""
    import oracle
    cores = oracle.default_threads()
    t0 = time.perf_counter()
    oracle.bwd_workload(wl.take_heads([0]), n_threads=cores)
    t1 = time.perf_counter() - t0
    heads = max(1, min(wl.H, int(target_seconds / max(t1, 1e-3))))
    if heads > 1:
        sub = wl.take_heads(list(range(heads)))
        t0 = time.perf_counter()
        oracle.bwd_workload(sub, n_threads=cores)
        t1 = time.perf_counter() - t0
    token_heads = wl.T_total * heads
    # tokens/s of the whole workload at this rate: all H heads of a token have to be processed
    value = (token_heads / t1) / wl.H
    sample = f"heads 0..{heads - 1} of {wl.name} ({token_heads} of {wl.T_total * wl.H} token-heads, {t1:.2f} s)"
    return value, cores, sample, min(cores, wl.N * heads)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2608_12700_b200 import synth
    wl = synth.config(args.config)
    vals = []
    for i in range(args.warmup + args.steps):
        per_step = max(1.0, min(args.cpu_seconds, 120.0 / max(1, args.warmup + args.steps)))
        v, cores, sample, used = time_oracle_sample(wl, per_step)
        if i >= args.warmup:
            vals.append(v)
    value = sum(vals) / len(vals)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * wl.tokens / value,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(wl),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2608_12700_b200 import benchutil, binding, runner, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the kernels")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    wl = synth.config(args.config)
    if rank:   # every rank its own batch of the same shape (heads permuted: chains are independent)
        import numpy as np
        rng = np.random.default_rng(1000 + rank)
        perm = rng.permutation(wl.H)
        wl = wl.take_heads(list(perm))
        wl.name = synth.CONFIG_NAMES[args.config]
    buf = runner.to_device(wl, dev)
    desc = buf.desc
    peaks = benchutil.load_peaks(ROOT)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---------------- device-resident timing ----------------
    for _ in range(max(3, args.warmup)):
        runner.run_bwd(buf)
    st = binding.gdn_last_device_status(buf.workspace)
    if st != binding.GDN_OK:
        raise binding.GdnError(st, "warm-up")
    sampler = benchutil.ClockSampler(local)
    # per-kernel durations are sampled inside the timed region: the kernels of every `period`-th step are bracketed
    # by events (an event between two kernels costs the stream a few microseconds; bracketing every launch slows a
    # 0.35 ms step by 5 %)
    period = max(1, args.steps // 12)
    binding.gdn_stage_timing_enable(period)
    binding.gdn_stage_timing_read()
    launches0 = binding.gdn_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    ev0.record(stream)
    for _ in range(args.steps):
        runner.run_bwd(buf)
    ev1.record(stream)
    barrier()
    sampler.stop()
    elapsed_ms = ev0.elapsed_time(ev1)
    launches = binding.gdn_launch_count() - launches0
    stages = binding.gdn_stage_timing_read()
    binding.gdn_stage_timing_enable(False)
    st = binding.gdn_last_device_status(buf.workspace)
    if st != binding.GDN_OK:
        raise binding.GdnError(st, "timed region")
    elapsed_ms, tokens_all = benchutil.aggregate_over_ranks(elapsed_ms, wl.tokens * args.steps, dist if world > 1 else None, dev)
    value = tokens_all / (elapsed_ms * 1e-3)
    ms_per_step = elapsed_ms / args.steps

    # ---------------- end to end: host buffers in, host buffers out ----------------
    # (the public host-buffer call: pinned host tensors in, pinned host tensors out; uploads, kernels and downloads of
    # independent pieces of the batch overlap inside it)
    host = None if args.no_e2e else runner.HostBackward(wl, dev)
    h2d = host.h2d_bytes if host else 0
    d2h = host.d2h_bytes if host else 0

    def e2e_step():
        host.step()

    e2e_steps = 0 if args.no_e2e else max(3, min(args.steps, 10))
    for _ in range(2 if e2e_steps else 0):
        e2e_step()
    barrier()
    ev0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    ev1.record(stream)
    barrier()
    if host:
        host.check()
    e2e_ms, e2e_tokens = benchutil.aggregate_over_ranks(ev0.elapsed_time(ev1), wl.tokens * e2e_steps, dist if world > 1 else None, dev)
    e2e_value = e2e_tokens / (e2e_ms * 1e-3) if e2e_steps else None

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---------------- roofline ----------------
    io_bytes = 2 if wl.dtype == "bf16" else 4
    token_heads, chains, chunk_heads = wl.T_total * wl.H, wl.N * wl.H, wl.n_chunks() * wl.H
    alg_bytes = benchutil.path_alg_bytes(token_heads=token_heads, chains=chains, d_k=wl.d_k, d_v=wl.d_v, io_bytes=io_bytes,
                                         delta_rule=wl.delta_rule, has_h0=wl.h0 is not None, has_dhT=wl.dhT is not None)
    alg_flops = benchutil.path_alg_flops(chunk_heads=chunk_heads, d_k=wl.d_k, d_v=wl.d_v, delta_rule=wl.delta_rule)
    t_hbm, t_tc = benchutil.roofline_times(alg_bytes, alg_flops, peaks, sustained=False)
    stage_ms = {k: v[0] / max(1, v[1]) for k, v in stages.items() if v[1] > 0}
    dom = max(stage_ms, key=stage_ms.get)
    # The dominant kernel is charged with the whole path's algorithmic work when it is the kernel that
    # streams the inputs and writes the gradients (the intra / fused gradient stage); a scan stage is
    # charged with the state traffic it cannot avoid.  Stated per stage in the design doc.
    dom_bytes, dom_flops = stage_algorithmic_work(dom, wl, io_bytes, binding.gdn_kernel_path(desc))
    d_hbm, d_tc = benchutil.roofline_times(dom_bytes, dom_flops, peaks, sustained=False)
    dom_s = stage_ms[dom] * 1e-3
    if d_hbm >= d_tc:
        roof = {"bound": "hbm", "achieved": dom_bytes / dom_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        roof = {"bound": "tensor", "achieved": dom_flops / dom_s / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = recorded_traffic(dom, wl)
    roof.update({"kernel": dom, "kernel_ms": stage_ms[dom], "peak_source": peaks["source"],
                 "algorithmic_bytes": dom_bytes, "algorithmic_flops": dom_flops})
    path_roof_s = max(t_hbm, t_tc)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
        "config": workload_config(wl),
        "kernel_path": binding.gdn_kernel_path(desc),
        "clocks": sampler.summary(),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms / max(1, e2e_steps), "steps": e2e_steps},
        "gpu_launches": launches,
        "roofline": roof,
        "path_roofline": {"algorithmic_bytes": alg_bytes, "algorithmic_flops": alg_flops, "t_hbm_us": t_hbm * 1e6,
                          "t_tensor_us": t_tc * 1e6, "bound": "hbm" if t_hbm >= t_tc else "tensor",
                          "frac": path_roof_s / (ms_per_step * 1e-3), "peak_source": peaks["source"]},
        "stage_ms_per_launch": {k: round(v, 5) for k, v in stage_ms.items()},
        "stage_timed_steps": max(v[1] for v in stages.values()),
    }
    if not args.no_cpu_baseline and world == 1:
        v, cores, sample, used = time_oracle_sample(wl, args.cpu_seconds)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def stage_algorithmic_work(stage, wl, io_bytes, family=""):
    """(bytes, flops) the named stage must move / multiply per launch (one launch covers the whole batch)."""
    from paper_2608_12700_b200 import benchutil
    th, chains, chd = wl.T_total * wl.H, wl.N * wl.H, wl.n_chunks() * wl.H
    dk, dv = wl.d_k, wl.d_v
    tri_k, tri_v, dense = 64 * 64 * dk, 64 * 64 * dv, 2 * 64 * dk * dv
    gates = 2 if wl.delta_rule else 1
    if family == "tcgen05_bf16_scalar_gate":
        # two fused passes per chain: the forward pass reads k, v, g; the backward pass streams every input and
        # writes every gradient (the whole path's algorithmic traffic) and runs 5 triangular + 4 dense products
        if stage == "fscan":
            return th * ((dk + dv) * io_bytes + 4), chd * dense
        if stage == "rscan":
            byts = benchutil.path_alg_bytes(token_heads=th, chains=chains, d_k=dk, d_v=dv, io_bytes=io_bytes, delta_rule=0,
                                            has_h0=False, has_dhT=wl.dhT is not None)
            return byts, chd * (3 * tri_k + 2 * tri_v + 4 * dense)
        return th * 4, 0.0
    if stage in ("fscan", "rscan", "scans"):
        # a carry stage must at least read its chunk-local operator and additive term and write one state per chunk;
        # "scans" is the launch that runs the forward and the reverse carry together
        ndir = 2 if stage == "scans" else 1
        return ndir * chd * (dk * dk + 2 * dk * dv) * io_bytes, ndir * chd * 2.0 * dk * dk * dv
    if stage == "prep":
        n_tri = 3 if family == "tcgen05_bf16" else 2
        return th * ((dk + dv) * io_bytes + 4 * gates), chd * (n_tri * tri_k + tri_v + 2 * dense + 2 * 64 ** 3 / 3)
    if stage == "eprep":
        return th * ((2 * dk + dv) * io_bytes), chd * (2 * tri_k + dense)
    # intra (or a fused gradient stage): streams every input and writes every gradient
    byts = benchutil.path_alg_bytes(token_heads=th, chains=chains, d_k=dk, d_v=dv, io_bytes=io_bytes,
                                    delta_rule=wl.delta_rule, has_h0=False, has_dhT=False, writes_dh0=False)
    # (in the tcgen05 d = 128 family P = tril(Q K^T . D) is formed by the prep stage and handed over: counted there)
    n_tri_k = 6 if family == "tcgen05_bf16" else 7
    flops = chd * ((n_tri_k * tri_k + 5 * tri_v + 5 * dense) if wl.delta_rule else (3 * tri_k + 2 * tri_v + 3 * dense))
    return byts, flops


def recorded_traffic(stage, wl):
    """DRAM bytes per launch of the stage from the ncu captures summarised under profiles/ (bytes per
    chunk-head measured on a small case, scaled by the chunk-heads of this workload), or None."""
    path = os.path.join(ROOT, "paper_2608_12700_b200", "measured_traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        rec = json.load(f)
    key = f"{stage}:{wl.dtype}:{wl.d_k}x{wl.d_v}:{wl.delta_rule}"
    if key not in rec:
        return None
    return rec[key]["bytes_per_chunk_head"] * wl.n_chunks() * wl.H


if __name__ == "__main__":
    a = parse()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
