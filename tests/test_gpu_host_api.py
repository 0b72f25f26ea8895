"""The host-buffer call: pieces of the batch are uploaded, processed and downloaded on overlapping streams; the
result must be the one of a single device-resident call, bit for bit, and correct against the oracle."""
import numpy as np
import pytest
import torch

from paper_2608_12700_b200 import runner, synth
from helpers import check_against_oracle

pytestmark = pytest.mark.gpu


def _as_f64(host_outputs):
    return {k: v.to(torch.float64).numpy() for k, v in host_outputs.items() if v is not None}


@pytest.mark.parametrize("case", ["d128_gdn", "d64_scalar_gate", "f32"])
@pytest.mark.parametrize("pieces", [None, 2, 1])
def test_pipelined_host_call_equals_device_call(case, pieces):
    kw = dict(d128_gdn=dict(dtype="bf16", B=4, T=200, H=2, d_k=128, d_v=128, states=True, seed=41),
              d64_scalar_gate=dict(dtype="bf16", B=4, T=200, H=2, d_k=64, d_v=64, delta_rule=0, g_scale=0.05, states=True, seed=42),
              f32=dict(dtype="f32", B=4, T=130, H=2, d_k=64, d_v=64, states=True, seed=43))[case]
    wl = synth.make_workload("host_" + case, **kw)
    ref = runner.backward(wl)
    host = runner.HostBackward(wl, pieces=pieces)
    for _ in range(2):            # twice: the second step reuses every buffer and event of the first
        for v in host.outputs.values():
            if v is not None:
                v.fill_(float("nan"))
        host.step()
        host.check()
        got = _as_f64(host.outputs)
        for name, r in ref.items():
            assert np.array_equal(got[name], r), (case, pieces, name)
    check_against_oracle(wl, got)


def test_packed_input_runs_as_one_piece():
    wl = synth.make_workload("host_packed", dtype="bf16", lengths=[65, 128, 0, 37, 300], H=2, d_k=128, d_v=128,
                             states=True, seed=44)
    host = runner.HostBackward(wl)
    assert host.pieces == 1
    host.step()
    host.check()
    check_against_oracle(wl, _as_f64(host.outputs))
