"""The tcgen05 d = 128 family carries the state across chunks in one of two forms: with the d x d operator of a
chunk (one product per step; chosen when few chains leave a step's latency exposed) or in low-rank form (two
dependent products per step, no operator: less HBM traffic; chosen when one CTA per chain and direction fills the
machine).  Both must reproduce the oracle on every kind of input; the shape decides only which one is faster."""
import numpy as np
import pytest

from paper_2608_12700_b200 import binding, runner, synth
from helpers import TOL, check_against_oracle, oracle_grads, rel

pytestmark = pytest.mark.gpu

OPERATOR, LOW_RANK = 2, 3   # arguments of gdn_debug_force_family

CASES = {
    "packed_ragged": dict(lengths=[200, 64, 75], H=2, states=True, seed=41),
    "equal_lengths": dict(B=2, T=256, H=3, states=True, seed=42),
    "short_sequences_no_states": dict(lengths=[1, 63, 65, 130], H=1, states=False, seed=43),
    "one_long_chain": dict(B=1, T=1100, H=1, states=True, seed=44),
    "with_empty_sequences": dict(lengths=[0, 70, 0, 130, 64, 0], H=2, states=True, seed=49),
}


@pytest.fixture
def carries(request):
    binding.gdn_debug_force_family(request.param)
    yield request.param
    binding.gdn_debug_force_family(0)


@pytest.mark.parametrize("carries", [OPERATOR, LOW_RANK], indirect=True)
@pytest.mark.parametrize("case", sorted(CASES))
def test_backward_matches_oracle_in_both_forms(case, carries):
    wl = synth.make_workload(f"carry_{case}", dtype="bf16", d_k=128, d_v=128, **CASES[case])
    buf = runner.to_device(wl)
    assert binding.gdn_kernel_path(buf.desc) == "tcgen05_bf16"
    runner.run_bwd(buf)
    check_against_oracle(wl, runner.fetch(buf))
    assert binding.gdn_last_device_status(buf.workspace) == binding.GDN_OK


@pytest.mark.parametrize("carries", [OPERATOR, LOW_RANK], indirect=True)
def test_forward_recompute_then_backward_on_its_workspace(carries):
    wl = synth.make_workload("carry_fwd", dtype="bf16", lengths=[70, 130, 64], H=2, d_k=128, d_v=128, states=True, seed=45)
    ref = oracle_grads(wl)
    buf = runner.to_device(wl, want_o=True)
    runner.run_fwd(buf)
    got = runner.fetch(buf)
    assert rel(got["o"], ref["o"]) < TOL["bf16"]
    assert rel(got["hT"], ref["hT"]) < TOL["bf16"]
    runner.run_bwd(buf, fresh=1)
    fresh = runner.fetch(buf)
    check_against_oracle(wl, fresh, ref=ref)
    whole = runner.backward(wl)   # the same form end to end: the same arithmetic, bit for bit
    for name in ("dq", "dk", "dv", "dg", "dbeta", "dh0"):
        assert np.array_equal(whole[name], fresh[name]), name


def test_forms_agree_with_each_other():
    """Both forms round the same quantities to bf16 at different places; they must agree far inside the tolerance."""
    wl = synth.make_workload("carry_agree", dtype="bf16", lengths=[300, 129], H=2, d_k=128, d_v=128, states=True, seed=46)
    out = {}
    try:
        for form in (OPERATOR, LOW_RANK):
            binding.gdn_debug_force_family(form)
            out[form] = runner.backward(wl)
    finally:
        binding.gdn_debug_force_family(0)
    for name in ("dq", "dk", "dv", "dg", "dbeta", "dh0"):
        assert rel(out[LOW_RANK][name], out[OPERATOR][name]) < 5e-3, name


def test_many_chains_choose_the_low_rank_form_by_themselves():
    """40 chains x 2 directions fill more than half of the machine with one CTA each: no override needed."""
    wl = synth.make_workload("carry_auto", dtype="bf16", B=10, T=130, H=4, d_k=128, d_v=128, states=True, seed=47)
    auto = runner.backward(wl)
    check_against_oracle(wl, auto)
    try:
        binding.gdn_debug_force_family(LOW_RANK)
        forced = runner.backward(wl)
    finally:
        binding.gdn_debug_force_family(0)
    for name in ("dq", "dk", "dv", "dg", "dbeta", "dh0"):
        assert np.array_equal(auto[name], forced[name]), name


def test_many_short_ragged_sequences_in_low_rank_form():
    """80 chains of 1 to 200 tokens: most chunks are ragged tails, many chains have a single step."""
    rng = np.random.default_rng(48)
    lengths = [int(x) for x in rng.integers(1, 201, size=40)]
    lengths[3], lengths[17] = 1, 64
    wl = synth.make_workload("carry_short", dtype="bf16", lengths=lengths, H=2, d_k=128, d_v=128, states=True, seed=48)
    check_against_oracle(wl, runner.backward(wl))
    buf = runner.to_device(wl, want_o=True)
    runner.run_fwd(buf)
    got, ref = runner.fetch(buf), oracle_grads(wl)
    assert rel(got["o"], ref["o"]) < TOL["bf16"]
    assert rel(got["hT"], ref["hT"]) < TOL["bf16"]


def test_operator_form_with_one_cta_per_chain():
    """With 40 chains the shape rule takes the low-rank form, and below 38 chains the operator form splits a chain over
    two CTAs; forcing the operator form here runs its one-CTA-per-(chain, direction) variant, which no shape selects by
    itself on a machine of this size."""
    wl = synth.make_workload("carry_operator_one_cta", dtype="bf16", B=1, T=192, H=40, d_k=128, d_v=128, states=True,
                             seed=50)
    try:
        binding.gdn_debug_force_family(OPERATOR)
        got = runner.backward(wl)
    finally:
        binding.gdn_debug_force_family(0)
    check_against_oracle(wl, got)
