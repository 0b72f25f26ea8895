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
    ap.add_argument("--no-others", action="store_true", help="skip the save-forward arm and the other configurations")
    ap.add_argument("--shape", default=None, metavar="B,T,H",
                    help="instead of a configuration: bf16 GDN, d_k = d_v = 128, B sequences of T tokens, H heads, with "
                         "states (value distributions of cfg1); used for kernel studies, not a bench line of its own")
    ap.add_argument("--carries", default="auto", choices=["auto", "operator", "lowrank"],
                    help="form of the inter-chunk carries of the tcgen05 d = 128 family (default: chosen by shape)")
    ap.add_argument("--channelwise", default=None, choices=["gdn", "kda", "gla"],
                    help="time gdn_bwd_channelwise (per-channel gate vectors; the named gate setting) on --shape "
                         "(default 4,2048,16) instead of the headline call; a kernel study, not the bench line")
    ap.add_argument("--arm", default="closed", choices=["closed", "save_forward"],
                    help="closed: gdn_bwd recomputes the forward (the headline); save_forward: every step is "
                         "gdn_fwd_recompute followed by gdn_bwd on its workspace (used when profiling that arm)")
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


def time_steps(fn, steps, barrier, stream):
    """Device time of `steps` back-to-back calls of fn, nothing but the calls between the two events."""
    import torch
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record(stream)
    for _ in range(steps):
        fn()
    ev1.record(stream)
    barrier()
    return ev0.elapsed_time(ev1)


def path_roofline(wl, peaks, ms_per_step):
    from paper_2608_12700_b200 import benchutil
    io_bytes = 2 if wl.dtype == "bf16" else 4
    alg_bytes = benchutil.path_alg_bytes(token_heads=wl.T_total * wl.H, chains=wl.N * wl.H, d_k=wl.d_k, d_v=wl.d_v,
                                         io_bytes=io_bytes, delta_rule=wl.delta_rule, has_h0=wl.h0 is not None,
                                         has_dhT=wl.dhT is not None)
    alg_flops = benchutil.path_alg_flops(chunk_heads=wl.n_chunks() * wl.H, d_k=wl.d_k, d_v=wl.d_v, delta_rule=wl.delta_rule)
    t_hbm, t_tc = benchutil.roofline_times(alg_bytes, alg_flops, peaks, sustained=False)
    return dict(algorithmic_bytes=alg_bytes, algorithmic_flops=alg_flops, t_hbm_us=t_hbm * 1e6, t_tensor_us=t_tc * 1e6,
                bound="hbm" if t_hbm >= t_tc else "tensor", frac=max(t_hbm, t_tc) / (ms_per_step * 1e-3),
                peak_source=peaks["source"])


def stage_pass(buf, runner, binding, calls, step=None):
    """Per-kernel durations from a separate, untimed-for-the-headline pass: every launch bracketed by events."""
    import torch
    binding.gdn_stage_timing_enable(1)
    binding.gdn_stage_timing_read()
    for _ in range(calls):
        step() if step else runner.run_bwd(buf)
    torch.cuda.synchronize()
    stages = binding.gdn_stage_timing_read()
    binding.gdn_stage_timing_enable(False)
    return {k: v[0] / v[1] for k, v in stages.items() if v[1] > 0}


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

    if args.shape:
        B_, T_, H_ = (int(x) for x in args.shape.split(","))
        wl = synth.make_workload(f"shape_B{B_}_T{T_}_H{H_}_bf16_d128", dtype="bf16", B=B_, T=T_, H=H_, d_k=128, d_v=128,
                                 seed=3, states=True)
    else:
        wl = synth.config(args.config)
    binding.gdn_debug_force_family({"auto": 0, "operator": 2, "lowrank": 3}[args.carries])
    if rank:   # every rank its own batch of the same shape (heads permuted: chains are independent)
        import numpy as np
        rng = np.random.default_rng(1000 + rank)
        perm = rng.permutation(wl.H)
        name = wl.name
        wl = wl.take_heads(list(perm))
        wl.name = name
    buf = runner.to_device(wl, dev)
    desc = buf.desc
    peaks = benchutil.load_peaks(ROOT)
    stream = torch.cuda.current_stream()
    warmup = max(3, args.warmup)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def check_status(b, where):
        st = binding.gdn_last_device_status(b.workspace)
        if st != binding.GDN_OK:
            raise binding.GdnError(st, where)

    # ---------------- device-resident timing: nothing but the K calls between the two events ----------------
    def step():
        if args.arm == "closed":
            runner.run_bwd(buf)
        else:
            runner.run_fwd(buf)
            runner.run_bwd(buf, fresh=1)

    for _ in range(warmup):
        step()
    check_status(buf, "warm-up")
    sampler = benchutil.ClockSampler(local, period_s=0.0005)
    launches0 = binding.gdn_launch_count()
    sampler.start()
    elapsed_ms = time_steps(step, args.steps, barrier, stream)
    sampler.stop()
    launches = binding.gdn_launch_count() - launches0
    check_status(buf, "timed region")
    elapsed_ms, tokens_all = benchutil.aggregate_over_ranks(elapsed_ms, wl.tokens * args.steps, dist if world > 1 else None, dev)
    value = tokens_all / (elapsed_ms * 1e-3)
    ms_per_step = elapsed_ms / args.steps

    # ---------------- per-kernel durations: a pass of its own, outside the headline ----------------
    stage_calls = max(3, min(args.steps, 10))
    stage_ms = stage_pass(buf, runner, binding, stage_calls, step)

    # ---------------- the arm that consumes a workspace saved by the forward (Section 4.5) ----------------
    save_forward = None
    if world == 1 and not args.no_others:
        runner.run_fwd(buf)
        for _ in range(warmup):
            runner.run_bwd(buf, fresh=1)
        sf_steps = max(3, min(args.steps, 20))
        sf_ms = time_steps(lambda: runner.run_bwd(buf, fresh=1), sf_steps, barrier, stream) / sf_steps
        fw_ms = time_steps(lambda: runner.run_fwd(buf), sf_steps, barrier, stream) / sf_steps
        check_status(buf, "save-forward arm")
        save_forward = {"ms_per_step": sf_ms, "tokens_per_s": wl.tokens / (sf_ms * 1e-3), "steps": sf_steps,
                        "gdn_fwd_recompute_ms": fw_ms,
                        "what": "gdn_bwd with workspace_is_fresh_from_fwd=1 on a workspace filled by gdn_fwd_recompute"}

    # ---------------- end to end: host buffers in, host buffers out ----------------
    # (the public host-buffer call: pinned host tensors in, pinned host tensors out; uploads, kernels and downloads of
    # independent pieces of the batch overlap inside it)
    host = None if args.no_e2e else runner.HostBackward(wl, dev)
    h2d = host.h2d_bytes if host else 0
    d2h = host.d2h_bytes if host else 0
    e2e_steps = 0 if args.no_e2e else max(3, min(args.steps, 10))
    for _ in range(2 if e2e_steps else 0):
        host.step()
    e2e_raw = time_steps(host.step, e2e_steps, barrier, stream) if e2e_steps else 0.0
    if host:
        host.check()
    e2e_ms, e2e_tokens = benchutil.aggregate_over_ranks(e2e_raw, wl.tokens * e2e_steps, dist if world > 1 else None, dev)
    e2e_value = e2e_tokens / (e2e_ms * 1e-3) if e2e_steps else None
    del host

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---------------- roofline: the whole path against its bound, the dominant kernel beside it ----------------
    io_bytes = 2 if wl.dtype == "bf16" else 4
    family = binding.gdn_kernel_path(desc)
    path = path_roofline(wl, peaks, ms_per_step)
    step_s = ms_per_step * 1e-3
    if path["bound"] == "hbm":
        roof = {"bound": "hbm", "achieved": path["algorithmic_bytes"] / step_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        roof = {"bound": "tensor", "achieved": path["algorithmic_flops"] / step_s / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    traffic = [recorded_traffic(k, wl, family, args.arm) for k in stage_ms]
    roof["traffic"] = sum(traffic) if traffic and all(t is not None for t in traffic) else None
    roof["traffic_over_algorithmic"] = roof["traffic"] / path["algorithmic_bytes"] if roof["traffic"] else None
    dom = max(stage_ms, key=stage_ms.get)
    dom_bytes, dom_flops = stage_algorithmic_work(dom, wl, io_bytes, family)
    d_hbm, d_tc = benchutil.roofline_times(dom_bytes, dom_flops, peaks, sustained=False)
    roof.update({
        "scope": "whole gdn_bwd call (all kernels of a step): algorithmic bytes of the path / ms_per_step; this is the "
                 "fraction the 50 % target is stated on",
        "peak_source": peaks["source"], "algorithmic_bytes": path["algorithmic_bytes"],
        "algorithmic_flops": path["algorithmic_flops"],
        "kernel": dom, "kernel_ms": stage_ms[dom], "kernel_algorithmic_bytes": dom_bytes,
        "kernel_algorithmic_flops": dom_flops, "kernel_traffic": recorded_traffic(dom, wl, family, args.arm),
        "kernel_frac": max(d_hbm, d_tc) / (stage_ms[dom] * 1e-3),
        "kernel_bound": "hbm" if d_hbm >= d_tc else "tensor"})
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
        "config": dict(workload_config(wl), arm=args.arm, carries=args.carries),
        "kernel_path": family,
        "clocks": sampler.summary(),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms / max(1, e2e_steps), "steps": e2e_steps},
        "gpu_launches": launches,
        "roofline": roof,
        "path_roofline": path,
        "stage_ms_per_launch": {k: round(v, 5) for k, v in stage_ms.items()},
        "stage_timed_calls": stage_calls,
    }
    if save_forward:
        line["save_forward_arm"] = save_forward
    del buf
    torch.cuda.empty_cache()
    binding.gdn_debug_force_family(0)
    if world == 1 and not args.no_others:
        line["other_configs"] = time_other_configs(args, peaks, barrier, stream, dev)
    if not args.no_cpu_baseline and world == 1:
        v, cores, sample, used = time_oracle_sample(wl, args.cpu_seconds)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_channelwise(args):
    """gdn_bwd_channelwise on one GPU: device-resident timing, per-kernel times, roofline of its own algorithmic bytes
    (q, k, v, dO and dq, dk, dv in bf16; g, b, dg, db [.., d_k] and w, dw [.., d_v] in fp32; states)."""
    import torch
    from paper_2608_12700_b200 import benchutil, binding, runner, synth
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    B_, T_, H_ = (int(x) for x in (args.shape or "4,2048,16").split(","))
    wl = synth.make_channelwise(f"channelwise_{args.channelwise}_bf16_B{B_}_T{T_}_H{H_}_d128", member=args.channelwise, dtype="bf16",
                                B=B_, T=T_, H=H_, d_k=128, d_v=128, seed=7, states=True)
    buf = runner.to_device_channelwise(wl, dev)
    stream = torch.cuda.current_stream()
    step = lambda: runner.run_bwd_channelwise(buf)
    for _ in range(max(3, args.warmup)):
        step()
    ms = time_steps(step, args.steps, torch.cuda.synchronize, stream) / args.steps
    st = binding.gdn_last_device_status(buf.workspace)
    if st != binding.GDN_OK:
        raise binding.GdnError(st, wl.name)
    stage_ms = stage_pass(buf, runner, binding, 3, step)
    peaks = benchutil.load_peaks(ROOT)
    th, chains = wl.T_total * wl.H, wl.N * wl.H
    alg = th * ((2 * 128 + 2 * 128) * 2 + (2 * 128 + 128) * 4 + (2 * 128 + 128) * 2 + (2 * 128 + 128) * 4) + chains * 3 * 128 * 128 * 4
    print(json.dumps({"metric": "gdn_bwd_channelwise_tokens_per_sec", "value": wl.tokens / (ms * 1e-3), "unit": UNIT,
                      "ms_per_step": ms, "steps": args.steps, "config": workload_config(wl),
                      "stage_ms_per_launch": {k: round(v, 5) for k, v in stage_ms.items()},
                      "roofline": {"bound": "hbm", "algorithmic_bytes": alg, "achieved": alg / (ms * 1e-3) / 1e9,
                                   "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": alg / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                   "peak_source": peaks["source"]}}))


def time_other_configs(args, peaks, barrier, stream, dev):
    """The other benchmark configurations, briefly (device-resident, same protocol as the headline), so that their
    figures come from the same run on the same machine.  Not bench lines of their own."""
    import torch
    from paper_2608_12700_b200 import binding, runner, synth
    out = {}
    # the five configurations, and the other shape of the paper's verification envelope (d_k = 128, d_v = 64; Section 4.5)
    # at the batch and length of the headline
    for idx in list(range(5)) + ["dk128_dv64"]:
        if idx == args.config:
            continue
        if idx == "dk128_dv64":
            wl = synth.make_workload("envelope_bf16_dk128_dv64", dtype="bf16", B=4, T=2048, H=16, d_k=128, d_v=64, seed=6, states=True)
        else:
            wl = synth.config(idx)
        buf = runner.to_device(wl, dev)
        for _ in range(3):
            runner.run_bwd(buf)
        steps = 20 if idx == 0 else 10
        ms = time_steps(lambda: runner.run_bwd(buf), steps, barrier, stream) / steps
        st = binding.gdn_last_device_status(buf.workspace)
        if st != binding.GDN_OK:
            raise binding.GdnError(st, wl.name)
        pr = path_roofline(wl, peaks, ms)
        stage_ms = stage_pass(buf, runner, binding, 3)
        out[wl.name] = {"ms_per_step": ms, "tokens_per_s": wl.tokens / (ms * 1e-3), "steps": steps, "tokens": wl.tokens,
                        "path_frac": pr["frac"], "path_bound": pr["bound"], "kernel_path": binding.gdn_kernel_path(buf.desc),
                        "stage_ms_per_launch": {k: round(v, 5) for k, v in stage_ms.items()}}
        del buf, wl
        torch.cuda.empty_cache()
    # the entry points with per-channel gates (tensor-core route): KDA gate setting on the shape of the headline
    wl = synth.make_channelwise("channelwise_kda_bf16_B4_T2048_H16_d128", member="kda", dtype="bf16", B=4, T=2048, H=16,
                                d_k=128, d_v=128, seed=7, states=True)
    buf = runner.to_device_channelwise(wl, dev)
    for _ in range(3):
        runner.run_bwd_channelwise(buf)
    ms = time_steps(lambda: runner.run_bwd_channelwise(buf), 10, barrier, stream) / 10
    st = binding.gdn_last_device_status(buf.workspace)
    if st != binding.GDN_OK:
        raise binding.GdnError(st, wl.name)
    binding.gdn_stage_timing_enable(1)
    binding.gdn_stage_timing_read()
    for _ in range(3):
        runner.run_bwd_channelwise(buf)
    torch.cuda.synchronize()
    stg = {k: round(v[0] / v[1], 5) for k, v in binding.gdn_stage_timing_read().items() if v[1] > 0}
    binding.gdn_stage_timing_enable(False)
    # the same backward on a workspace filled by the forward call, and that forward alone
    fwd_ms = time_steps(lambda: runner.run_fwd_channelwise(buf), 10, barrier, stream) / 10
    runner.run_fwd_channelwise(buf)
    fresh_ms = time_steps(lambda: runner.run_bwd_channelwise(buf, fresh=1), 10, barrier, stream) / 10
    out[wl.name] = {"ms_per_step": ms, "tokens_per_s": wl.tokens / (ms * 1e-3), "steps": 10, "tokens": wl.tokens,
                    "kernel_path": binding.gdn_kernel_path_channelwise(buf.desc), "entry_point": "gdn_bwd_channelwise",
                    "stage_ms_per_launch": stg,
                    "save_forward_arm": {"ms_per_step": fresh_ms, "gdn_fwd_recompute_channelwise_ms": fwd_ms}}
    del buf, wl
    torch.cuda.empty_cache()
    return out


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


def recorded_traffic(stage, wl, family="", arm="closed"):
    """DRAM bytes per launch of the stage from the ncu captures summarised under profiles/ (bytes per
    chunk-head measured on a small case, scaled by the chunk-heads of this workload), or None."""
    path = os.path.join(ROOT, "profiles", "measured_traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        rec = json.load(f)
    key = f"{stage}:{wl.dtype}:{wl.d_k}x{wl.d_v}:{wl.delta_rule}"
    if family == "tcgen05_bf16" and stage == "prep" and arm == "save_forward":
        key = f"factors:{wl.dtype}:{wl.d_k}x{wl.d_v}:{wl.delta_rule}"   # the forward's share of the preparation
    elif family == "tcgen05_bf16" and stage in ("prep", "scans"):
        from paper_2608_12700_b200 import binding, runner
        # the d = 128 family runs its carries in one of two forms with different traffic; the workspace size tells which
        desc = runner.desc_for(wl)
        per_ch = binding.gdn_workspace_bytes(desc)[1] / max(1, (wl.T_total // 64 + wl.N) * wl.H)
        if per_ch < 180 * 1024:
            key = f"{stage}_low_rank:{wl.dtype}:{wl.d_k}x{wl.d_v}:{wl.delta_rule}"
    if key not in rec:
        return None
    return rec[key]["bytes_per_chunk_head"] * wl.n_chunks() * wl.H


if __name__ == "__main__":
    a = parse()
    if a.impl == "reference":
        run_reference(a)
    elif a.channelwise:
        run_channelwise(a)
    else:
        run_ours(a)
