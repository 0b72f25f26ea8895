"""Several host threads, each with its own stream, workspace and problem, call the library at the same time: every result
must be bit-identical to the one the same problem gives alone.  (The library keeps no per-call state outside the
caller's workspace; its debug overrides are per thread.)"""
import threading

import numpy as np
import pytest
import torch

from paper_2608_12700_b200 import binding, runner, synth

pytestmark = pytest.mark.gpu

NAMES = ("dq", "dk", "dv", "dg", "dh0")


def problems():
    mk = synth.make_workload
    return [
        ("scalar", mk("thr_tc", dtype="bf16", lengths=[300, 64, 0, 129], H=3, d_k=128, d_v=128, states=True, seed=91)),
        ("scalar", mk("thr_tc_many", dtype="bf16", B=40, T=192, H=1, d_k=128, d_v=128, states=True, seed=92)),
        ("scalar", mk("thr_tc64", dtype="bf16", lengths=[200, 70], H=2, d_k=64, d_v=64, delta_rule=0, states=True, seed=93)),
        ("scalar", mk("thr_pad", dtype="bf16", B=2, T=130, H=2, d_k=128, d_v=64, states=True, seed=94)),
        ("scalar", mk("thr_f32", dtype="f32", lengths=[100, 30], H=2, d_k=64, d_v=64, states=True, seed=95)),
        ("channelwise", synth.make_channelwise("thr_cw", member="kda", dtype="bf16", lengths=[150, 64], H=2, d_k=128, d_v=128,
                                               states=True, seed=96)),
    ]


def run(kind, buf, stream):
    if kind == "scalar":
        runner.run_bwd(buf, stream=stream)
    else:
        runner.run_bwd_channelwise(buf, stream=stream)


def test_concurrent_callers_get_the_results_of_lone_callers():
    todo = problems()
    bufs = [runner.to_device(wl) if kind == "scalar" else runner.to_device_channelwise(wl) for kind, wl in todo]
    alone = []
    for (kind, wl), buf in zip(todo, bufs):
        run(kind, buf, None)
        alone.append(runner.fetch(buf))
    for buf in bufs:
        for t in buf.outputs.values():
            if t is not None:
                t.zero_()
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in todo]
    go = threading.Barrier(len(todo))
    errors = []

    def worker(i):
        try:
            torch.cuda.set_device(0)
            go.wait()
            for _ in range(25):
                run(todo[i][0], bufs[i], streams[i])
            streams[i].synchronize()
        except Exception as e:   # noqa: BLE001 (reported below)
            errors.append((i, repr(e)))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(len(todo))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    torch.cuda.synchronize()
    for (kind, wl), buf, ref in zip(todo, bufs, alone):
        assert binding.gdn_last_device_status(buf.workspace) == binding.GDN_OK, wl.name
        got = runner.fetch(buf)
        for n in NAMES + (("db", "dw") if kind == "channelwise" else ()):
            assert np.array_equal(got[n], ref[n]), (wl.name, n)
