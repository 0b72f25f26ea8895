"""Extreme gate settings through every kernel family against the oracle: no decay at all (g = 0: the pure delta rule),
decay so strong that a chunk's cumulative factor underflows fp32, erase / write gates at exactly 0 and exactly 1, and
tokens whose key is zero.  None of these may produce a non-finite value or leave the tolerance."""
import numpy as np
import pytest

from paper_2608_12700_b200 import runner, synth
from helpers import check_against_oracle

pytestmark = pytest.mark.gpu

FAMILIES = {
    "tcgen05_d128": dict(dtype="bf16", d_k=128, d_v=128, delta_rule=1),
    "tcgen05_d128_delta_off": dict(dtype="bf16", d_k=128, d_v=128, delta_rule=0),
    "tcgen05_padded": dict(dtype="bf16", d_k=128, d_v=64, delta_rule=1),
    "tcgen05_scalar_gate_d64": dict(dtype="bf16", d_k=64, d_v=64, delta_rule=0),
    "ffma_f32": dict(dtype="f32", d_k=64, d_v=64, delta_rule=1),
}


def workload(family, name, **kw):
    return synth.make_workload(f"{name}_{family}", lengths=[200, 64, 37], H=2, states=True, seed=120, scale=0.5,
                               **FAMILIES[family], **kw)


@pytest.mark.parametrize("family", FAMILIES)
def test_no_decay(family):
    wl = workload(family, "no_decay")
    wl.g[:] = 0.0
    check_against_oracle(wl, runner.backward(wl))


@pytest.mark.parametrize("family", FAMILIES)
@pytest.mark.parametrize("g_scale", [1.0, 4.0])
def test_strong_decay(family, g_scale):
    """g_scale 4: about -3.2 per token, -200 over a chunk: exp underflows to zero in fp32, the state is forgotten within
    a few tokens, and the gradient of the log decay is tiny but must still be right where it is not negligible."""
    wl = workload(family, f"decay_{g_scale}", g_scale=g_scale)
    check_against_oracle(wl, runner.backward(wl))


@pytest.mark.parametrize("family", [f for f in FAMILIES if FAMILIES[f]["delta_rule"]])
def test_gates_at_zero_and_one(family):
    wl = workload(family, "beta01")
    rng = np.random.default_rng(5)
    pick = rng.random(wl.beta.shape)
    wl.beta[pick < 0.3] = 0.0
    wl.beta[pick > 0.7] = 1.0
    check_against_oracle(wl, runner.backward(wl))


@pytest.mark.parametrize("family", FAMILIES)
def test_zero_keys(family):
    """Tokens whose key is the zero vector write nothing and erase nothing; a whole chunk of them leaves A = 0."""
    wl = workload(family, "zero_keys")
    wl.k[64:128] = 0.0                  # the second chunk of the first sequence
    wl.k[::7] = 0.0
    check_against_oracle(wl, runner.backward(wl))


# ---- the same regimes with per-channel gates ----
import oracle                                            # noqa: E402
from helpers import BLOCK_TOL, TOL, block_errors, rel    # noqa: E402

CW_FAMILIES = {
    "tcgen05_channelwise": dict(dtype="bf16", d_k=128, d_v=128),
    "tcgen05_channelwise_padded": dict(dtype="bf16", d_k=64, d_v=128),
    "ffma_f32_channelwise": dict(dtype="f32", d_k=64, d_v=64),
}


def cw_workload(family, name, **kw):
    return synth.make_channelwise(f"{name}_{family}", member="gdn", lengths=[200, 64, 37], H=2, states=True, seed=121, scale=0.5,
                                  **CW_FAMILIES[family], **kw)


def cw_check(wl):
    got = runner.backward_channelwise(wl)
    ref = oracle.vec_bwd_workload(wl)
    for n in ("dq", "dk", "dv", "dg", "db", "dw", "dh0"):
        assert np.all(np.isfinite(got[n])), n
        assert rel(got[n], ref[n]) <= TOL[wl.dtype], (wl.name, n, rel(got[n], ref[n]))
        e, _ = block_errors(wl, n, got[n], ref[n])
        assert e.size == 0 or e.max() <= BLOCK_TOL[wl.dtype], (wl.name, n, float(e.max()))


@pytest.mark.parametrize("family", CW_FAMILIES)
def test_channelwise_no_decay(family):
    wl = cw_workload(family, "cw_no_decay")
    wl.gv[:] = 0.0
    cw_check(wl)


@pytest.mark.parametrize("family", CW_FAMILIES)
def test_channelwise_decay_differs_by_orders_of_magnitude_between_channels(family):
    """Half of the key channels do not decay at all, the others lose a factor e^-60 per chunk (still inside the range the
    tensor-core route accepts): the per-channel scaling of keys and queries spans 26 orders of magnitude within a tile."""
    wl = cw_workload(family, "cw_mixed_decay")
    wl.gv[:, :, ::2] = 0.0
    wl.gv[:, :, 1::2] = -0.9
    cw_check(wl)


@pytest.mark.parametrize("family", CW_FAMILIES)
def test_channelwise_gates_at_zero_and_one_and_zero_keys(family):
    wl = cw_workload(family, "cw_01")
    rng = np.random.default_rng(6)
    for gate in (wl.bv, wl.wv):
        pick = rng.random(gate.shape)
        gate[pick < 0.3] = 0.0
        gate[pick > 0.7] = 1.0
    wl.k[64:128] = 0.0
    wl.k[::7] = 0.0
    cw_check(wl)
