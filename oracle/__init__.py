"""CPU fp64 oracle for the GDN backward -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke entry point and the benchmark's CPU-baseline leg may import this package.
It never imports the CUDA package and shares no code with it.

`build()` compiles `gdn_oracle.c` (one scalar gate triple per token and head) and `gdn_oracle_vec.c`
(the general recurrence with per-channel gate vectors) with gcc into `libgdn_oracle.so` next to this file;
`fwd()` / `bwd()` and `vec_fwd()` / `vec_bwd()` call them through ctypes with float64 numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gdn_oracle.c")
_SRC_VEC = os.path.join(_HERE, "gdn_oracle_vec.c")
_LIB = os.path.join(_HERE, "libgdn_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle (plain gcc, -O2, no fast-math so that fp64 rounding stays IEEE)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_SRC_VEC)):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fPIC", "-shared", "-std=c11", "-pthread", "-o", tmp, _SRC, _SRC_VEC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        P, I, D = ctypes.c_void_p, ctypes.c_int, ctypes.c_double
        lib.gdn_oracle_fwd.restype = I
        lib.gdn_oracle_fwd.argtypes = [I, P, I, I, I, D] + [P] * 9 + [I]
        lib.gdn_oracle_bwd.restype = I
        lib.gdn_oracle_bwd.argtypes = [I, P, I, I, I, D] + [P] * 18 + [I]
        lib.gdn_oracle_vec_fwd.restype = I
        lib.gdn_oracle_vec_fwd.argtypes = [I, P, I, I, I, D] + [P] * 9 + [I]
        lib.gdn_oracle_vec_bwd.restype = I
        lib.gdn_oracle_vec_bwd.argtypes = [I, P, I, I, I, D] + [P] * 18 + [I]
        _lib = lib
    return _lib


def _f64(a) -> Optional[np.ndarray]:
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def default_threads() -> int:
    return max(1, len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1))


def fwd(q, k, v, g, b, w, *, cu_seqlens, scale=1.0, h0=None, n_threads=None):
    """Token-serial forward.  Shapes: q,k [Tt,H,dk]; v [Tt,H,dv]; g,b,w [Tt,H]; h0 [N,H,dk,dv] or None.

    Returns (o [Tt,H,dv], hT [N,H,dk,dv]) as float64.
    """
    lib = _load()
    q, k, v, g, b, w, h0 = map(_f64, (q, k, v, g, b, w, h0))
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    Tt, H, dk = q.shape
    dv = v.shape[-1]
    N = len(cu) - 1
    assert int(cu[-1]) == Tt and k.shape == q.shape and v.shape[:2] == (Tt, H) and g.shape == (Tt, H)
    o = np.zeros((Tt, H, dv))
    hT = np.zeros((N, H, dk, dv))
    rc = lib.gdn_oracle_fwd(N, _ptr(cu), H, dk, dv, float(scale), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(b),
                            _ptr(w), _ptr(h0), _ptr(o), _ptr(hT), n_threads or default_threads())
    if rc != 0:
        raise RuntimeError(f"gdn_oracle_fwd failed with {rc}")
    return o, hT


def bwd(q, k, v, g, b, w, dO, *, cu_seqlens, scale=1.0, h0=None, dhT=None, n_threads=None):
    """Token-serial forward plus reverse-time adjoint of L = sum <dO,o> + <dhT,hT>.

    Returns a dict of float64 arrays: o, hT, dq, dk, dv, dg, db, dw, dh0.
    (For GDN, b = w = beta and d beta = db + dw.)
    """
    lib = _load()
    q, k, v, g, b, w, h0, dO, dhT = map(_f64, (q, k, v, g, b, w, h0, dO, dhT))
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    Tt, H, dk = q.shape
    dv = v.shape[-1]
    N = len(cu) - 1
    assert int(cu[-1]) == Tt and k.shape == q.shape and v.shape == dO.shape == (Tt, H, dv)
    out = dict(o=np.zeros((Tt, H, dv)), hT=np.zeros((N, H, dk, dv)), dq=np.zeros((Tt, H, dk)),
               dk=np.zeros((Tt, H, dk)), dv=np.zeros((Tt, H, dv)), dg=np.zeros((Tt, H)), db=np.zeros((Tt, H)),
               dw=np.zeros((Tt, H)), dh0=np.zeros((N, H, dk, dv)))
    rc = lib.gdn_oracle_bwd(N, _ptr(cu), H, dk, dv, float(scale), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(b),
                            _ptr(w), _ptr(h0), _ptr(dO), _ptr(dhT), _ptr(out["o"]), _ptr(out["hT"]),
                            _ptr(out["dq"]), _ptr(out["dk"]), _ptr(out["dv"]), _ptr(out["dg"]), _ptr(out["db"]),
                            _ptr(out["dw"]), _ptr(out["dh0"]), n_threads or default_threads())
    if rc != 0:
        raise RuntimeError(f"gdn_oracle_bwd failed with {rc}")
    return out


def bwd_workload(wl, n_threads=None):
    """Run the oracle on a synthetic workload object (fields q,k,v,dO,g,beta,h0,dhT,cu_seqlens,
    scale, delta_rule).  Gates: delta_rule=1 -> b = w = beta; delta_rule=0 -> b = 0, w = 1.
    Adds 'dbeta' = db + dw for the delta-rule case."""
    if wl.delta_rule:
        b = w = wl.beta
    else:
        b = np.zeros_like(wl.g)
        w = np.ones_like(wl.g)
    out = bwd(wl.q, wl.k, wl.v, wl.g, b, w, wl.dO, cu_seqlens=wl.cu_seqlens, scale=wl.scale, h0=wl.h0,
              dhT=wl.dhT, n_threads=n_threads)
    if wl.delta_rule:
        out["dbeta"] = out["db"] + out["dw"]
    return out


# ---- general recurrence with per-channel gates (gdn_oracle_vec.c) ----
def vec_fwd(q, k, v, g, b, w, *, cu_seqlens, scale=1.0, h0=None, n_threads=None):
    """Token-serial forward of Eq. 1 with gate vectors.  q,k,g,b [Tt,H,dk]; v,w [Tt,H,dv]; h0 [N,H,dk,dv] or None.
    Returns (o [Tt,H,dv], hT [N,H,dk,dv]) as float64."""
    lib = _load()
    q, k, v, g, b, w, h0 = map(_f64, (q, k, v, g, b, w, h0))
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    Tt, H, dk = q.shape
    dv = v.shape[-1]
    N = len(cu) - 1
    assert int(cu[-1]) == Tt and k.shape == g.shape == b.shape == q.shape and v.shape == w.shape == (Tt, H, dv)
    o = np.zeros((Tt, H, dv))
    hT = np.zeros((N, H, dk, dv))
    rc = lib.gdn_oracle_vec_fwd(N, _ptr(cu), H, dk, dv, float(scale), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(b),
                                _ptr(w), _ptr(h0), _ptr(o), _ptr(hT), n_threads or default_threads())
    if rc != 0:
        raise RuntimeError(f"gdn_oracle_vec_fwd failed with {rc}")
    return o, hT


def vec_bwd(q, k, v, g, b, w, dO, *, cu_seqlens, scale=1.0, h0=None, dhT=None, n_threads=None):
    """Forward plus reverse-time adjoint with gate vectors.  Returns float64 arrays o, hT, dq, dk, dv,
    dg [Tt,H,dk], db [Tt,H,dk], dw [Tt,H,dv], dh0."""
    lib = _load()
    q, k, v, g, b, w, h0, dO, dhT = map(_f64, (q, k, v, g, b, w, h0, dO, dhT))
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    Tt, H, dk = q.shape
    dv = v.shape[-1]
    N = len(cu) - 1
    assert int(cu[-1]) == Tt and k.shape == g.shape == b.shape == q.shape and v.shape == w.shape == dO.shape == (Tt, H, dv)
    out = dict(o=np.zeros((Tt, H, dv)), hT=np.zeros((N, H, dk, dv)), dq=np.zeros((Tt, H, dk)),
               dk=np.zeros((Tt, H, dk)), dv=np.zeros((Tt, H, dv)), dg=np.zeros((Tt, H, dk)), db=np.zeros((Tt, H, dk)),
               dw=np.zeros((Tt, H, dv)), dh0=np.zeros((N, H, dk, dv)))
    rc = lib.gdn_oracle_vec_bwd(N, _ptr(cu), H, dk, dv, float(scale), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(b),
                                _ptr(w), _ptr(h0), _ptr(dO), _ptr(dhT), _ptr(out["o"]), _ptr(out["hT"]),
                                _ptr(out["dq"]), _ptr(out["dk"]), _ptr(out["dv"]), _ptr(out["dg"]), _ptr(out["db"]),
                                _ptr(out["dw"]), _ptr(out["dh0"]), n_threads or default_threads())
    if rc != 0:
        raise RuntimeError(f"gdn_oracle_vec_bwd failed with {rc}")
    return out


def vec_bwd_workload(wl, n_threads=None):
    """Run the per-channel oracle on a synthetic channel-wise workload (fields q,k,v,dO,gv,bv,wv,h0,dhT,...)."""
    return vec_bwd(wl.q, wl.k, wl.v, wl.gv, wl.bv, wl.wv, wl.dO, cu_seqlens=wl.cu_seqlens, scale=wl.scale, h0=wl.h0,
                   dhT=wl.dhT, n_threads=n_threads)
