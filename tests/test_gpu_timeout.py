"""Failure detection on the device: every wait in the kernels is bounded, and a wait that runs out is reported
through the workspace's status word instead of hanging or trapping.  The test makes one wait run out on the host's
terms (a debugging hook shortens the limit to a millisecond for one call and has the first kernel leave out one of
its loads); nothing faults, and the same buffers give correct gradients on the next call."""
import numpy as np
import pytest
import torch

from paper_2608_12700_b200 import binding, runner, synth
from helpers import check_against_oracle

pytestmark = pytest.mark.gpu

GDN_ERR_DEVICE_TIMEOUT = 8


@pytest.mark.parametrize("lengths,H", [([64], 1), ([200, 64, 75], 2)])
def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_correct(lengths, H):
    wl = synth.make_workload("timeout", dtype="bf16", lengths=lengths, H=H, d_k=128, d_v=128, states=True, seed=90)
    buf = runner.to_device(wl)
    assert binding.gdn_kernel_path(buf.desc) == "tcgen05_bf16"
    for v in buf.outputs.values():
        if v is not None:
            v.fill_(7.0)
    binding.gdn_debug_inject_timeout(True)
    runner.run_bwd(buf)                                   # returns GDN_OK: the condition is only visible on the device
    assert binding.gdn_last_device_status(buf.workspace) == GDN_ERR_DEVICE_TIMEOUT
    assert "wait" in binding.status_string(GDN_ERR_DEVICE_TIMEOUT)
    # the stages after the one that gave up wrote nothing
    for n in ("dq", "dk", "dv", "dg", "dbeta"):
        assert torch.all(buf.outputs[n] == 7.0), n
    # the context is intact and the request was for one call: same buffers, same workspace, correct gradients
    runner.run_bwd(buf)
    check_against_oracle(wl, runner.fetch(buf))
    assert binding.gdn_last_device_status(buf.workspace) == binding.GDN_OK


def test_a_cancelled_request_changes_nothing():
    wl = synth.make_workload("timeout_cancel", dtype="bf16", lengths=[100], H=1, d_k=128, d_v=128, states=True, seed=91)
    binding.gdn_debug_inject_timeout(True)
    binding.gdn_debug_inject_timeout(False)
    check_against_oracle(wl, runner.backward(wl))
