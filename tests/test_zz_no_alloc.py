"""gdn_bwd_noalloc: the backward for callers that may not allocate device memory (frozen memory pools,
plug-ins that only receive input and output buffers).  It must give what gdn_bwd gives, call after call,
although every call reuses the same built-in scratch array.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from paper_2608_12700_b200 import binding, runner, synth
from helpers import TOL, rel

pytestmark = pytest.mark.gpu

NAMES = ("dq", "dk", "dv", "dg", "dbeta", "dh0")


def run_noalloc(buf):
    i, o = buf.inputs, buf.outputs
    binding.gdn_bwd_noalloc(buf.desc, i["q"], i["k"], i["v"], i["g"], i["beta"], i["h0"], i["dO"], i["dhT"],
                            i["cu_seqlens"], o["dq"], o["dk"], o["dv"], o["dg"], o["dbeta"], o["dh0"])
    torch.cuda.synchronize()
    return {n: o[n].detach().to(torch.float64).cpu().numpy() for n in NAMES}


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # two different problems back to back: the second call sees the first one's leftovers in the scratch
    first = synth.make_workload("noalloc_a", dtype="bf16", lengths=[200, 64, 75], H=2, d_k=128, d_v=128, seed=31, states=True)
    second = synth.make_workload("noalloc_b", dtype="f32", lengths=[130, 10], H=3, d_k=64, d_v=64, seed=32, states=True)
    for wl in (first, second):
        want = runner.backward(wl)                       # existing entry point, caller-provided workspace
        buf = runner.to_device(wl)
        for v in buf.outputs.values():
            if v is not None:
                v.fill_(float("nan"))
        got = run_noalloc(buf)
        for n in NAMES:
            assert np.isfinite(got[n]).all(), n
            assert rel(got[n], want[n]) <= TOL[wl.dtype], (wl.name, n, rel(got[n], want[n]))


def test_oversized_problem_is_refused_before_launch():
    desc = binding.make_desc(B=4, T=2048, H=16, d_k=128, d_v=128, N=4, dtype="bf16")
    _, need = binding.gdn_workspace_bytes(desc)
    assert need > binding.GDN_NOALLOC_WORKSPACE_BYTES
    dummy = torch.zeros(64, device="cuda")
    s = binding.gdn_bwd_noalloc(desc, dummy, dummy, dummy, dummy, dummy, None, dummy, None, None,
                                dummy, dummy, dummy, dummy, dummy, None, check=False)
    assert s == 6   # GDN_ERR_WORKSPACE_TOO_SMALL
