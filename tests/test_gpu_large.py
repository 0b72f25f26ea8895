"""Maximum sizes: tensors beyond 4 GiB (element offsets beyond 2^31, byte offsets beyond 2^32), hundreds of thousands
of chunk-heads, thousands of trips per persistent CTA.  Inputs are drawn on the device (too large to upload); the oracle
runs on chains copied back, chosen at the start, in the middle and at the very end of the tensors."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_12700_b200 import binding, runner, synth
from helpers import TOL, check_against_oracle, rel

pytestmark = pytest.mark.gpu

NEED_BYTES = 100e9


@pytest.mark.parametrize("case", ["d128_delta_rule", "d64_scalar_gate"])
def test_tensors_beyond_4_GiB(case):
    if torch.cuda.mem_get_info()[0] < NEED_BYTES:
        pytest.skip("needs about 90 GB of free device memory")
    if case == "d128_delta_rule":
        B, T, H, d, delta, family = 32, 16384, 40, 128, 1, "tcgen05_bf16"
    else:
        B, T, H, d, delta, family = 32, 32768, 40, 64, 0, "tcgen05_bf16_scalar_gate"
    assert B * T * H * d > 2 ** 31 and B * T * H * d * 2 > 2 ** 32
    dev = torch.device("cuda:0")
    inp = synth.device_inputs(B=B, T=T, H=H, d_k=d, d_v=d, dtype="bf16", seed=77, delta_rule=delta, states=True, device=dev)
    desc = binding.make_desc(B=B, T=T, H=H, d_k=d, d_v=d, N=B, dtype="bf16", scale=d ** -0.5, delta_rule=delta)
    assert binding.gdn_kernel_path(desc) == family
    ws = torch.empty(binding.gdn_workspace_bytes(desc)[1], dtype=torch.uint8, device=dev)
    out = dict(dq=torch.empty_like(inp["q"]), dk=torch.empty_like(inp["k"]), dv=torch.empty_like(inp["v"]),
               dg=torch.empty_like(inp["g"]), dbeta=torch.empty_like(inp["g"]) if delta else None,
               dh0=torch.empty_like(inp["h0"]))
    binding.gdn_bwd(desc, inp["q"], inp["k"], inp["v"], inp["g"], inp["beta"], inp["h0"], inp["dO"], inp["dhT"], None,
                    out["dq"], out["dk"], out["dv"], out["dg"], out["dbeta"], out["dh0"], ws)
    assert binding.gdn_last_device_status(ws) == binding.GDN_OK
    for name in ("dq", "dk", "dv"):   # nothing unwritten, nothing wild, anywhere in the tensors
        assert bool(torch.isfinite(out[name].view(-1)[:: 8191].float()).all()), name
    assert bool(torch.isfinite(out["dg"]).all()) and bool(torch.isfinite(out["dh0"]).all())

    host = lambda t, rows, hd: t[rows, hd:hd + 1].float().cpu().numpy().astype(np.float64)
    for n, hd in [(0, 0), (B // 2 + 1, 23), (B - 1, H - 1)]:
        rows = slice(n * T, (n + 1) * T)
        assert n == 0 or (n * T * H + hd) * d > 2 ** 31 // 2
        a = {x: host(inp[x], rows, hd) for x in ("q", "k", "v", "dO", "g")}
        beta = host(inp["beta"], rows, hd) if delta else None
        b = beta if delta else np.zeros_like(a["g"])
        w = beta if delta else np.ones_like(a["g"])
        st = lambda t: t[n:n + 1, hd:hd + 1].cpu().numpy().astype(np.float64)
        ref = oracle.bwd(a["q"], a["k"], a["v"], a["g"], b, w, a["dO"], cu_seqlens=np.array([0, T], np.int32),
                         scale=d ** -0.5, h0=st(inp["h0"]), dhT=st(inp["dhT"]))
        if delta:
            ref["dbeta"] = ref["db"] + ref["dw"]
        for name in ("dq", "dk", "dv", "dg") + (("dbeta",) if delta else ()):
            e = rel(host(out[name], rows, hd), ref[name])
            assert e <= TOL["bf16"], (case, n, hd, name, e)
        e = rel(st(out["dh0"]), ref["dh0"])
        assert e <= TOL["bf16"], (case, n, hd, "dh0", e)
    del inp, out, ws
    torch.cuda.empty_cache()


def test_sequence_longer_than_the_cached_chunk_decays():
    """The carry kernels keep the decays of a chain's first 2048 chunks in shared memory and read the later ones from
    the workspace: one sequence of 2049 chunks and a tail, in both forms of the carries, against the oracle (the oracle
    walks the 131 153 tokens serially: one call serves both)."""
    wl = synth.make_workload("long_chain", dtype="bf16", B=1, T=2049 * 64 + 17, H=2, d_k=128, d_v=128, states=True, seed=83,
                             g_scale=0.02, scale=128 ** -0.5)
    ref = oracle.bwd_workload(wl)
    for carries in (2, 3):
        binding.gdn_debug_force_family(carries)
        try:
            got = runner.backward(wl)
        finally:
            binding.gdn_debug_force_family(0)
        check_against_oracle(wl, got, ref=ref)
