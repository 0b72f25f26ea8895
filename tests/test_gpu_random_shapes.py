"""Seeded random descriptors through every entry point and kernel family, each against the oracle: lengths around chunk
borders, empty sequences, with and without states, fixed-length and packed, both dtypes, all head-dimension pairs, delta
rule on and off, scalar and per-channel gates.  What the hand-picked cases may have missed."""
import numpy as np
import pytest

import oracle
from paper_2608_12700_b200 import binding, runner, synth
from helpers import BLOCK_TOL, TOL, block_errors, check_against_oracle, rel

pytestmark = pytest.mark.gpu


def random_case(rng):
    dtype = "bf16" if rng.random() < 0.7 else "f32"
    dk, dv = (int(rng.choice([64, 128])) for _ in range(2))
    kw = dict(dtype=dtype, H=int(rng.integers(1, 6)), d_k=dk, d_v=dv, states=bool(rng.random() < 0.7),
              scale=float(rng.choice([1.0, 0.5, 0.088])), g_scale=float(rng.choice([0.02, 0.1, 0.3])))
    if rng.random() < 0.5:
        kw.update(B=int(rng.integers(1, 4)), T=int(rng.choice([1, 63, 64, 65, 127, 128, 129, 200, 333])))
    else:
        n = int(rng.integers(1, 7))
        kw.update(lengths=[int(rng.choice([0, 1, 17, 63, 64, 65, 100, 128, 130, 257])) for _ in range(n)])
    return kw


@pytest.mark.parametrize("seed", range(24))
def test_scalar_gates(seed):
    rng = np.random.default_rng(9000 + seed)
    kw = random_case(rng)
    kw["delta_rule"] = int(rng.random() < 0.7)
    wl = synth.make_workload(f"rand_{seed}", seed=9000 + seed, **kw)
    if wl.T_total == 0:
        kw["lengths"] = [70, 0]
        wl = synth.make_workload(f"rand_{seed}", seed=9000 + seed, **kw)
    buf = runner.to_device(wl, want_o=True)
    runner.run_bwd(buf)
    got = runner.fetch(buf)
    check_against_oracle(wl, got)
    runner.run_fwd(buf)
    f = runner.fetch(buf)
    ref = oracle.bwd_workload(wl)
    assert rel(f["o"], ref["o"]) < TOL[wl.dtype] and rel(f["hT"], ref["hT"]) < TOL[wl.dtype], binding.gdn_kernel_path(buf.desc)
    runner.run_bwd(buf, fresh=1)
    fresh = runner.fetch(buf)
    for n in ("dq", "dk", "dv", "dg", "dh0"):
        assert np.array_equal(fresh[n], got[n]), (n, binding.gdn_kernel_path(buf.desc))


@pytest.mark.parametrize("seed", range(12))
def test_channelwise_gates(seed):
    rng = np.random.default_rng(9500 + seed)
    kw = random_case(rng)
    if seed % 2 == 0:
        kw.update(dtype="bf16", d_k=128, d_v=128)           # the tensor-core route
    member = str(rng.choice(["gdn", "kda", "gla"]))
    wl = synth.make_channelwise(f"rand_cw_{seed}", member=member, seed=9500 + seed, **kw)
    if wl.T_total == 0:
        kw["lengths"] = [70, 0]
        wl = synth.make_channelwise(f"rand_cw_{seed}", member=member, seed=9500 + seed, **kw)
    got = runner.backward_channelwise(wl)
    ref = oracle.vec_bwd_workload(wl)
    for n in ("dq", "dk", "dv", "dg", "db", "dw", "dh0"):
        assert np.all(np.isfinite(got[n])), n
        if np.linalg.norm(ref[n]) == 0:
            # e.g. dg of one-token sequences without an initial state: the decay multiplies a zero state.  The tensor-core
            # route forms dg as a difference of products that cancel only up to rounding, so measure against their size.
            size = np.linalg.norm(ref["dq"].astype(np.float64) * wl.q) + np.linalg.norm(ref["dk"].astype(np.float64) * wl.k)
            assert np.linalg.norm(got[n]) <= TOL[wl.dtype] * max(size, 1e-30), (n, np.linalg.norm(got[n]), size)
            continue
        assert rel(got[n], ref[n]) <= TOL[wl.dtype], (wl.name, member, n, rel(got[n], ref[n]))
        e, _ = block_errors(wl, n, got[n], ref[n])
        assert e.size == 0 or e.max() <= BLOCK_TOL[wl.dtype], (wl.name, member, n, float(e.max()))


@pytest.mark.parametrize("dtype,d,delta", [("bf16", 128, 1), ("bf16", 64, 0), ("f32", 64, 1)])
def test_thousands_of_short_sequences(dtype, d, delta):
    """A packed batch of 3000 sequences of 0..150 tokens (many of them empty or shorter than a chunk): the chunk table,
    the chain-per-CTA carries and the persistent chunk kernels with far more chains than SMs."""
    rng = np.random.default_rng(4242)
    lengths = rng.integers(0, 151, size=3000)
    lengths[rng.random(3000) < 0.1] = 0
    wl = synth.make_workload(f"many_short_{dtype}_{d}", dtype=dtype, lengths=lengths.tolist(), H=2, d_k=d, d_v=d, states=True,
                             delta_rule=delta, seed=4243)
    got = runner.backward(wl)
    check_against_oracle(wl, got)
    empty = np.flatnonzero(lengths == 0)
    assert np.array_equal(got["dh0"][empty], wl.dhT[empty].astype(np.float64))   # empty sequences pass dhT through
