"""Thin ctypes binding of libgdn_b200.so: argument marshalling only.

Every function has the name and the argument order of its C counterpart (see include/gdn.h).  Tensors
are torch CUDA tensors used as plain device allocations; pointers, sizes and the current CUDA stream
are handed to the C ABI.  There is no fallback: if the library is missing or a call fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libgdn_b200.so")

GDN_OK = 0
GDN_F32, GDN_BF16 = 0, 1
STATUS_NAMES = {0: "GDN_OK", 1: "GDN_ERR_NULL_ARG", 2: "GDN_ERR_BAD_SHAPE", 3: "GDN_ERR_UNSUPPORTED_SHAPE",
                4: "GDN_ERR_MISALIGNED", 5: "GDN_ERR_BAD_SEQLENS", 6: "GDN_ERR_WORKSPACE_TOO_SMALL",
                7: "GDN_ERR_CUDA", 8: "GDN_ERR_DEVICE_TIMEOUT", 9: "GDN_ERR_DECAY_RANGE"}

EXPORTS = ["gdn_workspace_bytes", "gdn_fwd_recompute", "gdn_bwd", "gdn_last_device_status",
           "gdn_status_string", "gdn_kernel_path", "gdn_kernel_path_channelwise", "gdn_launch_count", "gdn_stage_timing_enable",
           "gdn_stage_timing_read", "gdn_debug_read", "gdn_debug_force_family", "gdn_bwd_noalloc",
           "gdn_noalloc_last_device_status", "gdn_workspace_bytes_channelwise", "gdn_fwd_recompute_channelwise",
           "gdn_bwd_channelwise", "gdn_debug_inject_timeout"]


class gdn_desc(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("T", ctypes.c_int32), ("H", ctypes.c_int32),
                ("d_k", ctypes.c_int32), ("d_v", ctypes.c_int32), ("chunk", ctypes.c_int32),
                ("N", ctypes.c_int32), ("dtype", ctypes.c_int32), ("scale", ctypes.c_float),
                ("delta_rule", ctypes.c_int32)]


class GdnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({status_string(status)})")


_lib = None


def lib():
    """Load the shared library; fails loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2608_12700_b200.build` "
                              "(there is no non-CUDA fallback)")
        L = ctypes.CDLL(LIB_PATH)
        P, I, Z = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
        D = ctypes.POINTER(gdn_desc)
        L.gdn_workspace_bytes.restype = I
        L.gdn_workspace_bytes.argtypes = [D, ctypes.POINTER(Z), ctypes.POINTER(Z)]
        L.gdn_fwd_recompute.restype = I
        L.gdn_fwd_recompute.argtypes = [D] + [P] * 9 + [P, Z, P]
        L.gdn_bwd.restype = I
        L.gdn_bwd.argtypes = [D] + [P] * 15 + [P, Z, I, P]
        L.gdn_last_device_status.restype = I
        L.gdn_last_device_status.argtypes = [P, P]
        L.gdn_status_string.restype = ctypes.c_char_p
        L.gdn_status_string.argtypes = [I]
        L.gdn_kernel_path.restype = ctypes.c_char_p
        L.gdn_kernel_path.argtypes = [D]
        L.gdn_kernel_path_channelwise.restype = ctypes.c_char_p
        L.gdn_kernel_path_channelwise.argtypes = [D]
        L.gdn_launch_count.restype = ctypes.c_uint64
        L.gdn_launch_count.argtypes = []
        L.gdn_stage_timing_enable.restype = I
        L.gdn_stage_timing_enable.argtypes = [I]
        L.gdn_stage_timing_read.restype = I
        L.gdn_stage_timing_read.argtypes = [I, P, P, P, P]
        L.gdn_bwd_noalloc.restype = I
        L.gdn_bwd_noalloc.argtypes = [D] + [P] * 15 + [P]
        L.gdn_workspace_bytes_channelwise.restype = I
        L.gdn_workspace_bytes_channelwise.argtypes = [D, ctypes.POINTER(Z), ctypes.POINTER(Z)]
        L.gdn_fwd_recompute_channelwise.restype = I
        L.gdn_fwd_recompute_channelwise.argtypes = [D] + [P] * 10 + [P, Z, P]
        L.gdn_bwd_channelwise.restype = I
        L.gdn_bwd_channelwise.argtypes = [D] + [P] * 17 + [P, Z, I, P]
        L.gdn_noalloc_last_device_status.restype = I
        L.gdn_noalloc_last_device_status.argtypes = [P]
        L.gdn_debug_read.restype = I
        L.gdn_debug_read.argtypes = [D, P, ctypes.c_char_p, I, I, P]
        L.gdn_debug_force_family.restype = I
        L.gdn_debug_force_family.argtypes = [I]
        L.gdn_debug_inject_timeout.restype = I
        L.gdn_debug_inject_timeout.argtypes = [I]
        _lib = L
    return _lib


def _p(t) -> Optional[int]:
    """Device (or host) address of a tensor, None for a missing optional argument."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def make_desc(*, B, T, H, d_k, d_v, N, dtype, scale=1.0, delta_rule=1, chunk=64) -> gdn_desc:
    code = {"f32": GDN_F32, "bf16": GDN_BF16}.get(dtype, dtype)
    return gdn_desc(B, T, H, d_k, d_v, chunk, N, code, scale, delta_rule)


def status_string(status: int) -> str:
    return lib().gdn_status_string(int(status)).decode()


def gdn_kernel_path(desc: gdn_desc) -> Optional[str]:
    r = lib().gdn_kernel_path(ctypes.byref(desc))
    return None if r is None else r.decode()


def gdn_kernel_path_channelwise(desc: gdn_desc) -> Optional[str]:
    r = lib().gdn_kernel_path_channelwise(ctypes.byref(desc))
    return None if r is None else r.decode()


def gdn_workspace_bytes(desc: gdn_desc):
    """Returns (fwd_bytes, bwd_bytes)."""
    f, b = ctypes.c_size_t(0), ctypes.c_size_t(0)
    s = lib().gdn_workspace_bytes(ctypes.byref(desc), ctypes.byref(f), ctypes.byref(b))
    if s != GDN_OK:
        raise GdnError(s, "gdn_workspace_bytes")
    return f.value, b.value


def gdn_fwd_recompute(desc, q, k, v, g, beta, h0, cu_seqlens, o, hT, workspace, workspace_bytes=None,
                      stream=None, check=True) -> int:
    wb = workspace.numel() * workspace.element_size() if workspace_bytes is None else workspace_bytes
    s = lib().gdn_fwd_recompute(ctypes.byref(desc), _p(q), _p(k), _p(v), _p(g), _p(beta), _p(h0), _p(cu_seqlens),
                                _p(o), _p(hT), _p(workspace), wb, _stream(stream))
    if check and s != GDN_OK:
        raise GdnError(s, "gdn_fwd_recompute")
    return s


def gdn_bwd(desc, q, k, v, g, beta, h0, dO, dhT, cu_seqlens, dq, dk, dv, dg, dbeta, dh0, workspace,
            workspace_bytes=None, workspace_is_fresh_from_fwd=0, stream=None, check=True) -> int:
    wb = workspace.numel() * workspace.element_size() if workspace_bytes is None else workspace_bytes
    s = lib().gdn_bwd(ctypes.byref(desc), _p(q), _p(k), _p(v), _p(g), _p(beta), _p(h0), _p(dO), _p(dhT),
                      _p(cu_seqlens), _p(dq), _p(dk), _p(dv), _p(dg), _p(dbeta), _p(dh0), _p(workspace), wb,
                      int(workspace_is_fresh_from_fwd), _stream(stream))
    if check and s != GDN_OK:
        raise GdnError(s, "gdn_bwd")
    return s


def gdn_last_device_status(workspace, stream=None) -> int:
    return lib().gdn_last_device_status(_p(workspace), _stream(stream))


def gdn_launch_count() -> int:
    return int(lib().gdn_launch_count())


def gdn_stage_timing_enable(on) -> None:
    """False/0: off.  True/1: every call's kernels are bracketed by events.  n > 1: every n-th call's."""
    lib().gdn_stage_timing_enable(int(on))


def gdn_stage_timing_read():
    """Returns {stage_name: (total_ms, launches)} accumulated since the previous read."""
    n = 32
    ms = (ctypes.c_float * n)()
    cnt = (ctypes.c_int32 * n)()
    names = (ctypes.c_char_p * n)()
    got = ctypes.c_int32(0)
    s = lib().gdn_stage_timing_read(n, ms, cnt, names, ctypes.byref(got))
    if s != GDN_OK:
        raise GdnError(s, "gdn_stage_timing_read")
    return {names[i].decode(): (float(ms[i]), int(cnt[i])) for i in range(got.value)}


def gdn_debug_force_family(family: int) -> None:
    """0: automatic dispatch.  1: FFMA kernels.  2 / 3: the tcgen05 d = 128 kernels carry the state across chunks
    in operator form / in low-rank form whatever the shape (by default the shape decides)."""
    s = lib().gdn_debug_force_family(int(family))
    if s != GDN_OK:
        raise GdnError(s, "gdn_debug_force_family")


def gdn_debug_read(desc: gdn_desc, workspace, what: str, chunk: int, head: int):
    """One workspace quantity of one (chunk, head) as a row-major float32 numpy array."""
    import numpy as np
    dk, dv = desc.d_k, desc.d_v
    shapes = {"gamma": (64,), "T": (64, 64), "W": (64, dk), "Ut": (64, dv), "Nm": (dk, dk), "Bf": (dk, dv),
              "hc": (dk, dv), "E": (dk, dv), "dhn": (dk, dv)}
    out = np.zeros(shapes[what], dtype=np.float32)
    s = lib().gdn_debug_read(ctypes.byref(desc), _p(workspace), what.encode(), int(chunk), int(head),
                             out.ctypes.data_as(ctypes.c_void_p))
    if s != GDN_OK:
        raise GdnError(s, "gdn_debug_read")
    return out


GDN_NOALLOC_WORKSPACE_BYTES = 32 * 1024 * 1024


def gdn_bwd_noalloc(desc, q, k, v, g, beta, h0, dO, dhT, cu_seqlens, dq, dk, dv, dg, dbeta, dh0, stream=None,
                    check=True) -> int:
    """gdn_bwd with the library's built-in scratch instead of a caller workspace (nothing is allocated)."""
    s = lib().gdn_bwd_noalloc(ctypes.byref(desc), _p(q), _p(k), _p(v), _p(g), _p(beta), _p(h0), _p(dO), _p(dhT),
                              _p(cu_seqlens), _p(dq), _p(dk), _p(dv), _p(dg), _p(dbeta), _p(dh0), _stream(stream))
    if check and s != GDN_OK:
        raise GdnError(s, "gdn_bwd_noalloc")
    return s


def gdn_noalloc_last_device_status(stream=None) -> int:
    """Device-side status of the last gdn_bwd_noalloc on the current device (synchronises the stream)."""
    return lib().gdn_noalloc_last_device_status(_stream(stream))


def gdn_workspace_bytes_channelwise(desc: gdn_desc):
    """Returns (fwd_bytes, bwd_bytes) of the channel-wise entry points."""
    f, b = ctypes.c_size_t(0), ctypes.c_size_t(0)
    s = lib().gdn_workspace_bytes_channelwise(ctypes.byref(desc), ctypes.byref(f), ctypes.byref(b))
    if s != GDN_OK:
        raise GdnError(s, "gdn_workspace_bytes_channelwise")
    return f.value, b.value


def gdn_fwd_recompute_channelwise(desc, q, k, v, g, b, w, h0, cu_seqlens, o, hT, workspace, workspace_bytes=None,
                                  stream=None, check=True) -> int:
    wb = workspace.numel() * workspace.element_size() if workspace_bytes is None else workspace_bytes
    s = lib().gdn_fwd_recompute_channelwise(ctypes.byref(desc), _p(q), _p(k), _p(v), _p(g), _p(b), _p(w), _p(h0),
                                            _p(cu_seqlens), _p(o), _p(hT), _p(workspace), wb, _stream(stream))
    if check and s != GDN_OK:
        raise GdnError(s, "gdn_fwd_recompute_channelwise")
    return s


def gdn_bwd_channelwise(desc, q, k, v, g, b, w, h0, dO, dhT, cu_seqlens, dq, dk, dv, dg, db, dw, dh0, workspace,
                        workspace_bytes=None, workspace_is_fresh_from_fwd=0, stream=None, check=True) -> int:
    wb = workspace.numel() * workspace.element_size() if workspace_bytes is None else workspace_bytes
    s = lib().gdn_bwd_channelwise(ctypes.byref(desc), _p(q), _p(k), _p(v), _p(g), _p(b), _p(w), _p(h0), _p(dO), _p(dhT),
                                  _p(cu_seqlens), _p(dq), _p(dk), _p(dv), _p(dg), _p(db), _p(dw), _p(dh0), _p(workspace),
                                  wb, int(workspace_is_fresh_from_fwd), _stream(stream))
    if check and s != GDN_OK:
        raise GdnError(s, "gdn_bwd_channelwise")
    return s


def gdn_debug_inject_timeout(on=True) -> None:
    """The next gdn_bwd of this thread on the tcgen05 d = 128 family makes one bounded device-side wait run out."""
    lib().gdn_debug_inject_timeout(1 if on else 0)
