"""CUDA-graph capture of the library calls: the calls allocate nothing, never synchronise and read no device value on
the host, so a stream capture records them; a replay must reproduce the eager result bit for bit."""
import numpy as np
import pytest
import torch

from paper_2608_12700_b200 import binding, runner, synth
from helpers import check_against_oracle

pytestmark = pytest.mark.gpu

CASES = {
    "tcgen05_d128": dict(dtype="bf16", lengths=[200, 64, 130], H=2, d_k=128, d_v=128, states=True, seed=31),
    "tcgen05_scalar_gate_d64": dict(dtype="bf16", lengths=[200, 64, 130], H=2, d_k=64, d_v=64, delta_rule=0,
                                    g_scale=0.05, states=True, seed=32),
    "ffma_f32": dict(dtype="f32", B=2, T=160, H=2, d_k=64, d_v=64, states=True, seed=33),
    "tcgen05_padded_dk128_dv64": dict(dtype="bf16", lengths=[200, 64, 130], H=2, d_k=128, d_v=64, states=True, seed=34),
    "tcgen05_d128_low_rank": dict(dtype="bf16", lengths=[70, 130, 64, 1, 100], H=8, d_k=128, d_v=128, states=True, seed=35),
}


def _snapshot(buf):
    torch.cuda.synchronize()
    return {k: v.clone() for k, v in buf.outputs.items() if v is not None}


def _clear(buf):
    for v in buf.outputs.values():
        if v is not None:
            v.fill_(float("nan") if v.is_floating_point() else 0)


@pytest.mark.parametrize("case", sorted(CASES))
def test_captured_backward_replays_bit_exact(case):
    wl = synth.make_workload("graph_" + case, **CASES[case])
    buf = runner.to_device(wl)
    runner.run_bwd(buf)                       # eager (also performs the one-time function attribute set-up)
    eager = _snapshot(buf)
    check_against_oracle(wl, runner.fetch(buf))

    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    _clear(buf)
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        runner.run_bwd(buf)                   # the binding passes the capturing (current) stream
    for _ in range(3):
        _clear(buf)
        graph.replay()
        got = _snapshot(buf)
        for name, ref in eager.items():
            assert torch.equal(got[name].view(torch.uint8), ref.view(torch.uint8)), (case, name)
    assert binding.gdn_last_device_status(buf.workspace) == binding.GDN_OK


def test_captured_forward_then_backward_on_its_workspace():
    """Forward recompute and the backward that consumes its workspace, recorded as one graph."""
    wl = synth.make_workload("graph_fwd_bwd", **CASES["tcgen05_d128"])
    buf = runner.to_device(wl, want_o=True)
    runner.run_fwd(buf)
    runner.run_bwd(buf, fresh=1)
    eager = _snapshot(buf)

    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        runner.run_fwd(buf)
        runner.run_bwd(buf, fresh=1)
    _clear(buf)
    graph.replay()
    got = _snapshot(buf)
    for name, ref in eager.items():
        assert torch.equal(got[name].view(torch.uint8), ref.view(torch.uint8)), name
    assert binding.gdn_last_device_status(buf.workspace) == binding.GDN_OK
    assert np.isfinite(got["o"].float().cpu().numpy()).all()


@pytest.mark.parametrize("dk", [64, 128])   # FFMA kernels / tensor-core route
def test_captured_channelwise_backward_replays_bit_exact(dk):
    wl = synth.make_channelwise("graph_channelwise", member="kda", dtype="bf16", lengths=[100, 64, 30], H=2, d_k=dk, d_v=128,
                                states=True, seed=36)
    buf = runner.to_device_channelwise(wl)
    runner.run_bwd_channelwise(buf)
    eager = _snapshot(buf)
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    _clear(buf)
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        runner.run_bwd_channelwise(buf)
    for _ in range(2):
        _clear(buf)
        graph.replay()
        got = _snapshot(buf)
        for name, ref in eager.items():
            assert torch.equal(got[name].view(torch.uint8), ref.view(torch.uint8)), name
    assert binding.gdn_last_device_status(buf.workspace) == binding.GDN_OK
