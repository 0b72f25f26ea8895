"""gdn_bwd_noalloc: the backward for callers that may not allocate device memory (frozen memory pools,
plug-ins that only receive input and output buffers).  It must give what gdn_bwd gives, bit for bit, call
after call, although every call reuses the same built-in scratch array and finds the previous call's
leftovers in it.  Collected last on purpose: a run that stops at the first failure has then already run
every other test.  Nothing here depends on what ran before it."""
import numpy as np
import pytest
import torch

from paper_2608_12700_b200 import binding, runner, synth

pytestmark = pytest.mark.gpu

NAMES = ("dq", "dk", "dv", "dg", "dbeta", "dh0")


def run_noalloc(buf, fetch=True):
    i, o = buf.inputs, buf.outputs
    binding.gdn_bwd_noalloc(buf.desc, i["q"], i["k"], i["v"], i["g"], i["beta"], i["h0"], i["dO"], i["dhT"],
                            i["cu_seqlens"], o["dq"], o["dk"], o["dv"], o["dg"], o["dbeta"], o["dh0"])
    torch.cuda.synchronize()
    if not fetch:
        return None
    return {n: o[n].detach().to(torch.float64).cpu().numpy() for n in NAMES if o[n] is not None}


def problems():
    mk = synth.make_workload
    return [
        # fp32 FFMA family first, so that every tile-image family below starts on a dirty array
        mk("noalloc_f32", dtype="f32", lengths=[130, 10], H=3, d_k=64, d_v=64, seed=32, states=True),
        # bf16 d = 128, few chains: carries in operator form, two CTAs per chain
        mk("noalloc_operator", dtype="bf16", lengths=[200, 64, 75], H=2, d_k=128, d_v=128, seed=31, states=True),
        # non-finite input: its leftovers in the array are poison for whoever reads before writing
        mk("noalloc_poison", dtype="bf16", lengths=[100, 90], H=2, d_k=128, d_v=128, seed=36, states=True),
        # 40 chains: carries in low-rank form, ragged tails
        mk("noalloc_lowrank", dtype="bf16", lengths=[70, 130, 64, 1, 100], H=8, d_k=128, d_v=128, seed=33, states=True),
        # scalar-gate family (d = 64, delta rule off), ragged, with states
        mk("noalloc_scalar_gate", dtype="bf16", lengths=[65, 128, 0, 37, 300], H=3, d_k=64, d_v=64, delta_rule=0,
           g_scale=0.05, seed=34, states=True),
        mk("noalloc_f32_again", dtype="f32", B=2, T=100, H=2, d_k=64, d_v=128, seed=35, states=True),
    ]


def test_calls_in_a_row_match_the_workspace_entry_point_bit_for_bit():
    expected_paths = {"noalloc_operator": "tcgen05_bf16", "noalloc_lowrank": "tcgen05_bf16",
                      "noalloc_scalar_gate": "tcgen05_bf16_scalar_gate"}
    for wl in problems():
        if wl.name == "noalloc_poison":
            wl.v[50, 1, 7] = np.nan
            wl.dO[120, 0, 3] = np.inf
        want = runner.backward(wl)                       # existing entry point, caller-provided workspace
        buf = runner.to_device(wl)
        if wl.name in expected_paths:
            assert binding.gdn_kernel_path(buf.desc) == expected_paths[wl.name]
        for v in buf.outputs.values():
            if v is not None:
                v.fill_(float("nan"))
        got = run_noalloc(buf)
        assert binding.gdn_noalloc_last_device_status() == binding.GDN_OK
        for n in got:
            # the same deterministic kernels on the same inputs: equal bit patterns (NaNs included)
            assert np.array_equal(got[n], want[n], equal_nan=True), (wl.name, n)
            if wl.name != "noalloc_poison":
                assert np.isfinite(got[n]).all(), (wl.name, n)


def test_a_second_call_allocates_no_device_memory():
    wl = problems()[3]
    buf = runner.to_device(wl)
    run_noalloc(buf)                                     # first call on the device: address look-up, module load
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    run_noalloc(buf, fetch=False)                        # (no tensor conversions either: torch's allocator stays idle)
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before                     # device memory as the driver sees it: nothing taken, nothing returned


def test_oversized_problem_is_refused_before_launch():
    desc = binding.make_desc(B=4, T=2048, H=16, d_k=128, d_v=128, N=4, dtype="bf16")
    _, need = binding.gdn_workspace_bytes(desc)
    assert need > binding.GDN_NOALLOC_WORKSPACE_BYTES
    dummy = torch.zeros(64, device="cuda")
    s = binding.gdn_bwd_noalloc(desc, dummy, dummy, dummy, dummy, dummy, None, dummy, None, None,
                                dummy, dummy, dummy, dummy, dummy, None, check=False)
    assert s == 6   # GDN_ERR_WORKSPACE_TOO_SMALL


def test_argument_errors_are_refused_before_anything_is_enqueued():
    wl = problems()[0]
    buf = runner.to_device(wl)
    i, o = buf.inputs, buf.outputs
    launches = binding.gdn_launch_count()
    s = binding.gdn_bwd_noalloc(buf.desc, i["q"], i["k"], None, i["g"], i["beta"], i["h0"], i["dO"], i["dhT"],
                                i["cu_seqlens"], o["dq"], o["dk"], o["dv"], o["dg"], o["dbeta"], o["dh0"], check=False)
    assert s == 1   # GDN_ERR_NULL_ARG
    assert binding.gdn_launch_count() == launches


def test_malformed_cu_seqlens_is_visible_through_the_status_reader():
    """A data error that only the device can see: the call returns GDN_OK, the kernels stop early, and the status
    word of the built-in scratch says why.  The next well-formed call clears it."""
    wl = problems()[0]
    buf = runner.to_device(wl)
    good = buf.inputs["cu_seqlens"]
    buf.inputs["cu_seqlens"] = torch.tensor([0, 135, 130], dtype=torch.int32, device="cuda")   # decreasing
    run_noalloc(buf)
    assert binding.gdn_noalloc_last_device_status() == 5   # GDN_ERR_BAD_SEQLENS
    buf.inputs["cu_seqlens"] = good
    run_noalloc(buf)
    assert binding.gdn_noalloc_last_device_status() == binding.GDN_OK
