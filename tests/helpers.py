"""Shared helpers for the GPU parity tests: run the CUDA path through the C ABI and the oracle on the
same seeded inputs and compare per gradient tensor (normwise relative error over valid tokens), then
block by block (one 64-token chunk of one head) so that a single wrong chunk or tail cannot hide in a
large tensor."""
import numpy as np

import oracle

TOL = {"f32": 1e-4, "bf16": 2e-2}          # per-gradient-tensor normwise relative error bounds (the acceptance bound)
# Per-block bound: normwise error of one (64-token chunk, head) block -- one (sequence, head) state for dh0 --
# relative to that block's oracle norm, floored at a tenth of the tensor's root-mean-square block norm (a block
# that happens to be nearly zero is measured against the typical block, not against itself).  A block is
# 64 x d values (64 for the gate gradients), so its error fluctuates around the tensor's; a wrong block reads ~1.
BLOCK_TOL = {"f32": 1e-3, "bf16": 5e-2}
GRADS = ("dq", "dk", "dv", "dg", "dbeta", "dh0")


def rel(a, b):
    a = np.asarray(a, dtype=np.float64); b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a - b))


def oracle_grads(wl):
    return oracle.bwd_workload(wl)


def chunk_starts(wl):
    """First token of every 64-token chunk of every sequence (chunks never straddle a sequence border)."""
    cu = np.asarray(wl.cu_seqlens, dtype=np.int64)
    starts = [np.arange(cu[n], cu[n + 1], wl.chunk) for n in range(len(cu) - 1)]
    return np.concatenate(starts) if starts else np.zeros(0, dtype=np.int64)


def block_errors(wl, name, got, ref):
    """Normwise error of every block of one gradient tensor, each relative to max(own oracle norm, floor).
    Returns (errors [n_blocks, H], floor)."""
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    if name == "dh0":
        d2 = ((got - ref) ** 2).sum(axis=(2, 3)); r2 = (ref ** 2).sum(axis=(2, 3))          # [N, H]
    else:
        st = chunk_starts(wl)
        if got.shape[0] == 0 or len(st) == 0:
            return np.zeros((0, got.shape[1])), 0.0
        sq = lambda x: (x ** 2).reshape(x.shape[0], x.shape[1], -1).sum(axis=2)            # [Tt, H]
        d2 = np.add.reduceat(sq(got - ref), st, axis=0); r2 = np.add.reduceat(sq(ref), st, axis=0)
    floor = 0.1 * np.sqrt(r2.mean()) if r2.size else 0.0
    den = np.maximum(np.sqrt(r2), floor)
    with np.errstate(invalid="ignore", divide="ignore"):
        e = np.where(den > 0, np.sqrt(d2) / den, np.sqrt(d2))
    return e, floor


def check_against_oracle(wl, got, tol=None, names=GRADS, ref=None, block_tol=None):
    """Returns {name: error}; asserts each tensor is finite and within tolerance as a whole (the acceptance
    bound) and block by block (BLOCK_TOL)."""
    tol = TOL[wl.dtype] if tol is None else tol
    block_tol = BLOCK_TOL[wl.dtype] if block_tol is None else block_tol
    ref = oracle_grads(wl) if ref is None else ref
    errs, worst = {}, {}
    for n in names:
        if n == "dbeta" and not wl.delta_rule:
            continue
        assert np.all(np.isfinite(got[n])), f"{n} has non-finite values"
        errs[n] = rel(got[n], ref[n])
        e, _ = block_errors(wl, n, got[n], ref[n])
        if e.size:
            i = np.unravel_index(np.argmax(e), e.shape)
            worst[n] = (float(e[i]), tuple(int(x) for x in i))
    bad = {n: e for n, e in errs.items() if not e <= tol}
    assert not bad, f"{wl.name}: over tolerance {tol}: {bad} (all: {errs})"
    badb = {n: w for n, w in worst.items() if not w[0] <= block_tol}
    assert not badb, f"{wl.name}: blocks over {block_tol} (error, (block, head)): {badb} (whole tensors: {errs})"
    errs["worst_block"] = max((w[0] for w in worst.values()), default=0.0)
    return errs
