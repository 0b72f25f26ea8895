"""Stored values: the figures the paper prints for this path (as bounds) and a lock on the oracle's own outputs."""
import json
import os

import numpy as np

import oracle
from oracle import chunked
from paper_2608_12700_b200 import synth

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _figures():
    with open(os.path.join(GOLDEN, "paper_figures.json")) as f:
        return json.load(f)


def test_oracle_reproduces_its_stored_outputs():
    """oracle_tiny.json was written by tests/golden/make_oracle_golden.py from `oracle/` alone; any change of the
    oracle's arithmetic shows up here (differences beyond a few ulps of fp64)."""
    with open(os.path.join(GOLDEN, "oracle_tiny.json")) as f:
        gold = json.load(f)
    for name, rec in gold["cases"].items():
        wl = synth.make_workload("golden_" + name, **rec["args"])
        res = oracle.bwd_workload(wl, n_threads=1)
        assert set(res) == set(rec["outputs"]), name
        for k, stored in rec["outputs"].items():
            now = np.asarray(res[k], dtype=np.float64).ravel()
            ref = np.asarray(stored, dtype=np.float64)
            assert now.shape == ref.shape, (name, k)
            scale = max(1.0, float(np.abs(ref).max()))
            assert float(np.abs(now - ref).max()) <= 1e-13 * scale, (name, k)


def test_chunked_form_agrees_with_the_recurrence_within_the_papers_fp64_bound():
    """The paper's double-precision cross-check bound (Section 4.5) applied to this build's two CPU rungs: the
    chunkwise fp64 formulation against the token-serial oracle, per gradient tensor, normwise."""
    bound = _figures()["fp64_crosscheck_bound"]["value"]
    for seed, extra in ((7, {}), (8, dict(delta_rule=0, g_scale=0.05))):
        wl = synth.make_workload("fig_bound", dtype="f32", lengths=[130, 64, 37], H=2, d_k=16, d_v=8, states=True,
                                 seed=seed, **extra)
        ref = oracle.bwd_workload(wl)
        if wl.delta_rule:
            b = w = wl.beta
        else:
            b, w = np.zeros_like(wl.g), np.ones_like(wl.g)
        got = chunked.bwd(wl.q, wl.k, wl.v, wl.g, b, w, wl.dO, cu_seqlens=wl.cu_seqlens, scale=wl.scale, h0=wl.h0,
                          dhT=wl.dhT)
        for k in ("o", "hT", "dq", "dk", "dv", "dg", "db", "dw", "dh0"):
            den = np.linalg.norm(ref[k])
            err = np.linalg.norm(np.asarray(got[k]) - ref[k]) / (den if den > 0 else 1.0)
            assert err <= bound, (k, err)
