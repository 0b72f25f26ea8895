"""Shared helpers for the GPU parity tests: run the CUDA path through the C ABI and the oracle on the
same seeded inputs and compare per gradient tensor (normwise relative error over valid tokens)."""
import numpy as np

import oracle

TOL = {"f32": 1e-4, "bf16": 2e-2}   # per-gradient-tensor normwise relative error bounds
GRADS = ("dq", "dk", "dv", "dg", "dbeta", "dh0")


def rel(a, b):
    a = np.asarray(a, dtype=np.float64); b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a - b))


def oracle_grads(wl):
    return oracle.bwd_workload(wl)


def check_against_oracle(wl, got, tol=None, names=GRADS, ref=None):
    """Returns {name: error}; asserts each is within tolerance and finite."""
    tol = TOL[wl.dtype] if tol is None else tol
    ref = oracle_grads(wl) if ref is None else ref
    errs = {}
    for n in names:
        if n == "dbeta" and not wl.delta_rule:
            continue
        assert np.all(np.isfinite(got[n])), f"{n} has non-finite values"
        errs[n] = rel(got[n], ref[n])
    bad = {n: e for n, e in errs.items() if not e <= tol}
    assert not bad, f"{wl.name}: over tolerance {tol}: {bad} (all: {errs})"
    return errs
