"""Writes tests/golden/oracle_tiny.json: a tiny seeded problem with the oracle's outputs, as a lock against accidental
changes of the oracle's arithmetic.  Calls only `oracle/` and the seeded input generator.

    python tests/golden/make_oracle_golden.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2608_12700_b200 import synth  # noqa: E402

CASES = {
    # two sequences (one crossing a chunk border, one shorter than a chunk), two heads, states on both ends
    "gdn": dict(dtype="f32", lengths=[65, 3], H=1, d_k=4, d_v=3, states=True, seed=2024, scale=0.7),
    # delta rule off: b = 0, w = 1
    "scalar_gate": dict(dtype="f32", lengths=[66], H=1, d_k=2, d_v=3, states=True, seed=2025, delta_rule=0, g_scale=0.05),
}


def main():
    out = {"_what": "oracle outputs (fp64, repr round-trips exactly) for synth.make_workload(name, **args)", "cases": {}}
    for name, args in CASES.items():
        wl = synth.make_workload("golden_" + name, **args)
        res = oracle.bwd_workload(wl, n_threads=1)   # forward outputs o, hT and every gradient
        out["cases"][name] = {"args": args,
                              "outputs": {k: np.asarray(v, dtype=np.float64).ravel().tolist() for k, v in res.items()}}
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_tiny.json")
    with open(path, "w") as f:
        json.dump(out, f)
    print("wrote", path, os.path.getsize(path), "bytes")


if __name__ == "__main__":
    main()
