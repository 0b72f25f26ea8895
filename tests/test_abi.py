"""Host-side checks of the C ABI: the library loads, exports every function include/gdn.h declares, and
rejects bad arguments on the host before touching a GPU."""
import ctypes
import os
import re

import pytest

from paper_2608_12700_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gdn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gdn_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"gdn_workspace_bytes", "gdn_fwd_recompute", "gdn_bwd", "gdn_last_device_status", "gdn_status_string"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(binding.EXPORTS) == set(names)


def test_status_strings(lib):
    for code in range(10):
        assert binding.status_string(code)
    assert "unknown" in binding.status_string(99)


def test_workspace_sizes_and_shape_errors(lib):
    ok = binding.make_desc(B=4, T=2048, H=16, d_k=128, d_v=128, N=4, dtype="bf16")
    f, b = binding.gdn_workspace_bytes(ok)
    assert 0 < f <= b
    for bad, code in [(dict(d_k=96), 3), (dict(chunk=32), 3), (dict(H=0), 2), (dict(dtype=7), 3), (dict(delta_rule=2), 2)]:
        kw = dict(B=1, T=64, H=1, d_k=64, d_v=64, N=1, dtype="f32")
        kw.update(bad)
        d = binding.make_desc(**kw)
        with pytest.raises(binding.GdnError) as e:
            binding.gdn_workspace_bytes(d)
        assert e.value.status == code


def test_pointer_errors_are_caught_on_the_host(lib):
    d = binding.make_desc(B=1, T=64, H=1, d_k=64, d_v=64, N=1, dtype="f32")
    _, need = binding.gdn_workspace_bytes(d)
    A = 4096   # fake, aligned, never dereferenced: every check below fails before any launch
    args = dict(q=A, k=A, v=A, g=A, beta=A, h0=None, dO=A, dhT=None, cu_seqlens=None, dq=A, dk=A, dv=A, dg=A, dbeta=A, dh0=None)

    def call(ws=A, wb=need, **over):
        a = dict(args); a.update(over)
        return binding.lib().gdn_bwd(ctypes.byref(d), a["q"], a["k"], a["v"], a["g"], a["beta"], a["h0"], a["dO"], a["dhT"],
                                     a["cu_seqlens"], a["dq"], a["dk"], a["dv"], a["dg"], a["dbeta"], a["dh0"], ws, wb, 0, None)

    assert call(q=None) == 1                 # GDN_ERR_NULL_ARG
    assert call(dbeta=None) == 1             # required for the delta rule
    assert call(ws=None) == 1
    assert call(k=A + 2) == 4                # GDN_ERR_MISALIGNED
    assert call(wb=need - 1) == 6            # GDN_ERR_WORKSPACE_TOO_SMALL
    d2 = binding.make_desc(B=2, T=64, H=1, d_k=64, d_v=64, N=2, dtype="f32")
    assert binding.lib().gdn_bwd(ctypes.byref(d2), A, A, A, A, A, None, A, None, A, A, A, A, A, A, None, A, 1 << 40, 0, None) == 2
    d3 = binding.make_desc(B=2, T=64, H=1, d_k=64, d_v=64, N=3, dtype="f32")
    assert binding.lib().gdn_bwd(ctypes.byref(d3), A, A, A, A, A, None, A, None, None, A, A, A, A, A, None, A, 1 << 40, 0, None) == 2


def test_kernel_family_names(lib):
    assert binding.gdn_kernel_path(binding.make_desc(B=1, T=64, H=1, d_k=128, d_v=128, N=1, dtype="bf16")) == "tcgen05_bf16"
    assert binding.gdn_kernel_path(binding.make_desc(B=1, T=64, H=1, d_k=64, d_v=64, N=1, dtype="f32")) == "simt_f32"
