"""GPU parity of the entry points with per-channel gates (Eq. 1 with gate vectors; KDA, GLA and the full GDN as
gate settings, Table 2) against the per-channel CPU fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_12700_b200 import binding, runner, synth
from helpers import BLOCK_TOL, TOL, block_errors, rel

pytestmark = pytest.mark.gpu

GRADS = ("dq", "dk", "dv", "dg", "db", "dw", "dh0")


def check(wl, got, names=GRADS):
    ref = oracle.vec_bwd_workload(wl)
    errs = {}
    for n in names:
        assert np.all(np.isfinite(got[n])), n
        errs[n] = rel(got[n], ref[n])
        e, _ = block_errors(wl, n, got[n], ref[n])
        if e.size:
            assert e.max() <= BLOCK_TOL[wl.dtype], (wl.name, n, "block", float(e.max()))
    bad = {n: e for n, e in errs.items() if not e <= TOL[wl.dtype]}
    assert not bad, f"{wl.name}: over tolerance: {bad} (all: {errs})"
    return errs, ref


@pytest.mark.parametrize("member", ["gdn", "kda", "gla"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_family_members_ragged_with_states(dtype, member):
    # a tail of 1, an exact multiple, an empty sequence, a sub-chunk sequence, a long ragged one
    wl = synth.make_channelwise(f"cw_{member}_{dtype}", member=member, dtype=dtype, lengths=[65, 128, 0, 37, 300], H=2,
                                d_k=64, d_v=64, states=True, seed=61, scale=0.5)
    got = runner.backward_channelwise(wl)
    errs, _ = check(wl, got)
    print(wl.name, errs)
    assert np.array_equal(got["dh0"][2], wl.dhT[2].astype(np.float64))   # empty sequence: pass-through


@pytest.mark.parametrize("member", ["gdn", "kda", "gla"])
def test_tensor_core_carries_bf16_d128(member):
    """bf16 I/O at d_k = d_v = 128: the forward and the reverse carry (K#1) run on the tcgen05 kernels, fed with tile
    images by the preparation kernels; ragged, with states and an empty sequence; forward outputs and the
    save-forward arm as well."""
    wl = synth.make_channelwise(f"cw_tc_{member}", member=member, dtype="bf16", lengths=[65, 128, 0, 37, 300], H=2,
                                d_k=128, d_v=128, states=True, seed=68, scale=0.5)
    got = runner.backward_channelwise(wl)
    errs, ref = check(wl, got)
    print(wl.name, errs)
    assert np.array_equal(got["dh0"][2], wl.dhT[2].astype(np.float64))
    buf = runner.to_device_channelwise(wl, want_o=True)
    runner.run_fwd_channelwise(buf)
    f = runner.fetch(buf)
    assert rel(f["o"], ref["o"]) < TOL["bf16"] and rel(f["hT"], ref["hT"]) < TOL["bf16"]
    runner.run_bwd_channelwise(buf, fresh=1)
    fresh = runner.fetch(buf)
    for n in GRADS:
        assert np.array_equal(fresh[n], got[n]), n


@pytest.mark.parametrize("dk,dv", [(128, 128), (128, 64), (64, 128)])
def test_shapes(dk, dv):
    wl = synth.make_channelwise(f"cw_shape_{dk}_{dv}", dtype="f32", B=2, T=192, H=2, d_k=dk, d_v=dv, states=True, seed=62)
    check(wl, runner.backward_channelwise(wl))


def test_forward_outputs_and_fresh_workspace():
    wl = synth.make_channelwise("cw_fwd", dtype="f32", lengths=[70, 130], H=2, d_k=64, d_v=64, states=True, seed=63)
    buf = runner.to_device_channelwise(wl, want_o=True)
    runner.run_fwd_channelwise(buf)
    got = runner.fetch(buf)
    ref = oracle.vec_bwd_workload(wl)
    assert rel(got["o"], ref["o"]) < TOL["f32"] and rel(got["hT"], ref["hT"]) < TOL["f32"]
    runner.run_bwd_channelwise(buf, fresh=1)
    fresh = runner.fetch(buf)
    whole = runner.backward_channelwise(wl)
    for n in GRADS:
        assert np.array_equal(whole[n], fresh[n]), n


def test_equal_entries_agree_with_the_scalar_gate_entry_point():
    """Gate vectors with equal entries are the scalar-gate problem: dq, dk, dv, dh0 agree with gdn_bwd and the gate
    gradients are its channel sums (Appendix A: the scalar path recovers only channel sums)."""
    sc = synth.make_workload("cw_vs_scalar", dtype="f32", lengths=[100, 64, 30], H=2, d_k=64, d_v=64, states=True, seed=64)
    want = runner.backward(sc)
    wl = synth.make_workload("cw_vs_scalar", dtype="f32", lengths=[100, 64, 30], H=2, d_k=64, d_v=64, states=True, seed=64)
    wl.gv = np.ascontiguousarray(np.repeat(sc.g[:, :, None], 64, axis=2))
    wl.bv = np.ascontiguousarray(np.repeat(sc.beta[:, :, None], 64, axis=2))
    wl.wv = np.ascontiguousarray(np.repeat(sc.beta[:, :, None], 64, axis=2))
    got = runner.backward_channelwise(wl)
    for n in ("dq", "dk", "dv", "dh0"):
        assert rel(got[n], want[n]) < 1e-5, n
    assert rel(got["dg"].sum(-1), want["dg"]) < 1e-4
    assert rel(got["db"].sum(-1) + got["dw"].sum(-1), want["dbeta"]) < 1e-4


def test_erase_gate_zero_makes_the_solve_vanish_bitwise():
    wl = synth.make_channelwise("cw_gla_T", member="gla", dtype="f32", B=1, T=128, H=2, d_k=64, d_v=64, seed=65)
    buf = runner.to_device_channelwise(wl)
    runner.run_bwd_channelwise(buf)
    assert binding.gdn_last_device_status(buf.workspace) == 0
    # T sits behind the per-channel gamma block in this family's workspace: find it through the sizes
    ch_heads = (wl.T_total // 64 + wl.N) * wl.H
    off = 256
    for n in (wl.N + 1, wl.T_total // 64 + wl.N, wl.T_total // 64 + wl.N, wl.T_total // 64 + wl.N):
        off += (4 * n + 255) // 256 * 256
    off += (4 * ch_heads * 64 * 64 + 255) // 256 * 256          # gamma [CH, 64, d_k]
    T = buf.workspace[off:off + 4 * 64 * 64 * 4].view(torch.float32).reshape(4, 64, 64).cpu().numpy()
    for t in T:
        assert np.array_equal(t, np.eye(64, dtype=np.float32))


def test_bitwise_determinism_and_untouched_inputs():
    wl = synth.make_channelwise("cw_det", dtype="bf16", lengths=[100, 260], H=2, d_k=128, d_v=128, states=True, seed=66)
    buf = runner.to_device_channelwise(wl)
    before = {k: v.clone() for k, v in buf.inputs.items() if v is not None}
    runner.run_bwd_channelwise(buf)
    first = {k: v.clone() for k, v in buf.outputs.items() if v is not None}
    for _ in range(2):
        for v in buf.outputs.values():
            if v is not None:
                v.fill_(float("nan"))
        runner.run_bwd_channelwise(buf)
        torch.cuda.synchronize()
        for k, v in first.items():
            assert torch.equal(v.view(torch.uint8), buf.outputs[k].view(torch.uint8)), k
    for k, v in before.items():
        assert torch.equal(v, buf.inputs[k]), k
    check(wl, runner.fetch(buf))


def test_argument_errors():
    wl = synth.make_channelwise("cw_err", dtype="f32", B=1, T=64, H=1, d_k=64, d_v=64, seed=67)
    buf = runner.to_device_channelwise(wl)
    i, o = buf.inputs, buf.outputs
    s = binding.gdn_bwd_channelwise(buf.desc, i["q"], i["k"], i["v"], i["g"], None, i["w"], None, i["dO"], None, None,
                                    o["dq"], o["dk"], o["dv"], o["dg"], o["db"], o["dw"], None, buf.workspace, check=False)
    assert s == 1
    s = binding.gdn_bwd_channelwise(buf.desc, i["q"], i["k"], i["v"], i["g"], i["b"], i["w"], None, i["dO"], None, None,
                                    o["dq"], o["dk"], o["dv"], o["dg"], o["db"], o["dw"], None, buf.workspace,
                                    workspace_bytes=1024, check=False)
    assert s == 6


def test_decay_beyond_the_range_of_the_tensor_core_route_falls_back_on_the_device():
    """bf16 I/O at d = 128 scales keys by exp(-gam), which is only safe while the cumulative log decay of a chunk stays in
    [-80, 80].  A call whose gates leave that range is computed by the FFMA kernels instead (the decision is taken on the
    device: the tensor-core kernels stand down, the fall-back launches behind them do the work) and must be just as
    right; the status word ends up clean, and the next call with tame gates is back on the tensor cores."""
    wl = synth.make_channelwise("cw_range", dtype="bf16", lengths=[100, 64], H=2, d_k=128, d_v=128, states=True, seed=69)
    wl.gv[70:100, 1, 5] = -3.0                       # channel 5 of head 1: 30 tokens of e^-3 inside the second chunk
    buf = runner.to_device_channelwise(wl, want_o=True)
    for v in buf.outputs.values():
        if v is not None:
            v.fill_(float("nan"))
    runner.run_bwd_channelwise(buf)
    assert binding.gdn_last_device_status(buf.workspace) == binding.GDN_OK
    errs, ref = check(wl, runner.fetch(buf))
    assert max(errs[n] for n in ("dg", "db", "dw", "dh0")) < 1e-5     # fp32 arithmetic on that route (dq, dk, dv are bf16)
    # forward outputs and the save-forward arm take the same decision
    runner.run_fwd_channelwise(buf)
    f = runner.fetch(buf)
    assert rel(f["o"], ref["o"]) < TOL["bf16"] and rel(f["hT"], ref["hT"]) < 1e-5
    # (the workspace then holds the fall-back kernels' fp32 data, which its header remembers: the backward that consumes it
    # must run on them as well, whatever its own launches would prefer)
    runner.run_bwd_channelwise(buf, fresh=1)
    errs, _ = check(wl, runner.fetch(buf))
    assert max(errs[n] for n in ("dg", "db", "dw", "dh0")) < 1e-5
    # tame gates again: tensor-core route, bf16-level errors in the gate gradients; closed arm, then forward + save-forward arm
    wl.gv[70:100, 1, 5] = -0.1
    buf.inputs["g"].copy_(torch.from_numpy(wl.gv))
    runner.run_bwd_channelwise(buf)
    closed = runner.fetch(buf)
    errs, _ = check(wl, closed)
    assert errs["dg"] > 1e-4
    runner.run_fwd_channelwise(buf)
    runner.run_bwd_channelwise(buf, fresh=1)
    fresh = runner.fetch(buf)
    for n in GRADS:
        assert np.array_equal(fresh[n], closed[n]), n


def test_tensor_core_route_with_several_trips_per_cta_and_equal_lengths():
    """More chunk-heads than SMs (every persistent CTA makes at least two trips, some three) and a fixed-length batch
    (no cu_seqlens): both the look-ahead loads and the arithmetic chunk geometry are exercised."""
    wl = synth.make_channelwise("cw_trips", member="gdn", dtype="bf16", B=3, T=700, H=10, d_k=128, d_v=128, states=True, seed=70)
    assert (wl.T_total // 64 + 3) * wl.H > 2 * torch.cuda.get_device_properties(0).multi_processor_count
    errs, _ = check(wl, runner.backward_channelwise(wl))
    print(wl.name, errs)


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("f32", 64)])
def test_no_tokens_passes_the_state_gradient_through(dtype, d):
    wl = synth.make_channelwise("cw_empty", dtype=dtype, lengths=[0, 0], H=2, d_k=d, d_v=d, states=True, seed=71)
    got = runner.backward_channelwise(wl)
    assert np.array_equal(got["dh0"], wl.dhT.astype(np.float64))


@pytest.mark.parametrize("member", ["gdn", "kda"])
@pytest.mark.parametrize("dk,dv", [(128, 64), (64, 128), (64, 64)])
def test_head_dimension_64_is_padded_onto_the_tensor_core_route(dk, dv, member):
    """bf16 I/O with a head dimension of 64: inputs, gate vectors and states are zero-padded to d = 128 inside the
    workspace and the tcgen05 kernels run (a padded key channel has decay 1 and erase gate 0, a padded value channel
    write gate 0: every product is what it was).  Against the oracle, with the forward outputs and the save-forward
    arm; the FFMA family on the same inputs must agree with the oracle too."""
    wl = synth.make_channelwise(f"cw_pad_{dk}_{dv}_{member}", member=member, dtype="bf16", lengths=[65, 128, 0, 37, 300], H=3,
                                d_k=dk, d_v=dv, states=True, seed=71, scale=0.5)
    buf = runner.to_device_channelwise(wl, want_o=True)
    assert binding.gdn_kernel_path_channelwise(buf.desc) == "tcgen05_bf16_channelwise_padded"
    runner.run_bwd_channelwise(buf)
    got = runner.fetch(buf)
    errs, ref = check(wl, got)
    print(wl.name, errs)
    assert np.array_equal(got["dh0"][2], wl.dhT[2].astype(np.float64))
    runner.run_fwd_channelwise(buf)
    f = runner.fetch(buf)
    assert rel(f["o"], ref["o"]) < TOL["bf16"] and rel(f["hT"], ref["hT"]) < TOL["bf16"]
    runner.run_bwd_channelwise(buf, fresh=1)
    fresh = runner.fetch(buf)
    for n in GRADS:
        assert np.array_equal(fresh[n], got[n]), n
    binding.gdn_debug_force_family(1)
    try:
        fbuf = runner.to_device_channelwise(wl)
        assert binding.gdn_kernel_path_channelwise(fbuf.desc) == "simt_bf16_channelwise"
        runner.run_bwd_channelwise(fbuf)
        check(wl, runner.fetch(fbuf))
    finally:
        binding.gdn_debug_force_family(0)


def test_kernel_path_names():
    mk = lambda dt, dk, dv: binding.make_desc(B=1, T=64, H=1, d_k=dk, d_v=dv, N=1, dtype=dt)
    assert binding.gdn_kernel_path_channelwise(mk("bf16", 128, 128)) == "tcgen05_bf16_channelwise"
    assert binding.gdn_kernel_path_channelwise(mk("bf16", 64, 64)) == "tcgen05_bf16_channelwise_padded"
    assert binding.gdn_kernel_path_channelwise(mk("f32", 128, 128)) == "simt_f32_channelwise"


def test_full_size_shape_of_the_bench_every_chain():
    """The workload `bench.py` times for the channel-wise calls (KDA gates, bf16, B = 4, T = 2048, H = 16, d = 128; 2048
    chunk-heads, 14 trips per persistent CTA), every chain against the per-channel oracle, whole tensors and 64-token
    blocks."""
    wl = synth.make_channelwise("channelwise_kda_bf16_B4_T2048_H16_d128", member="kda", dtype="bf16", B=4, T=2048, H=16,
                                d_k=128, d_v=128, seed=7, states=True)
    errs, _ = check(wl, runner.backward_channelwise(wl))
    print(wl.name, errs)
