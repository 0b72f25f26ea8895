"""Persistent-kernel edge cases of the tcgen05 families: numbers of chunk-heads around the number of SMs (a CTA makes
zero, one or two trips; the last trip of some CTAs has no successor to load for), and the number of chains around the
point where the carries switch from the operator form (two CTAs per chain and direction) to the low-rank form."""
import numpy as np
import pytest
import torch

from paper_2608_12700_b200 import runner, synth
from helpers import check_against_oracle

pytestmark = pytest.mark.gpu


def _sms():
    return torch.cuda.get_device_properties(0).multi_processor_count


@pytest.mark.parametrize("delta", [-1, 0, 1])
@pytest.mark.parametrize("trips", [1, 2])
def test_chunk_heads_around_a_multiple_of_the_sm_count(trips, delta):
    heads = trips * _sms() + delta          # one chunk per head: chunk-heads = heads
    wl = synth.make_workload(f"edge_{trips}_{delta}", dtype="bf16", B=1, T=64, H=heads, d_k=128, d_v=128, states=True,
                             seed=500 + 10 * trips + delta)
    check_against_oracle(wl, runner.backward(wl))


def test_single_chunk_head_and_ragged_single_token():
    for lengths in ([64], [1], [63], [65]):
        wl = synth.make_workload("edge_single_%d" % lengths[0], dtype="bf16", lengths=lengths, H=1, d_k=128, d_v=128,
                                 states=True, seed=600 + lengths[0])
        check_against_oracle(wl, runner.backward(wl))


@pytest.mark.parametrize("chains", [36, 37, 38, 74, 75])
def test_scan_variants_around_their_switch_over(chains):
    # the operator form with a chain's state columns split over two CTAs is used while 4 x chains CTAs fit the SMs;
    # beyond that the carries take the low-rank form with one CTA per (chain, direction)
    wl = synth.make_workload(f"edge_scan_{chains}", dtype="bf16", B=1, T=192, H=chains, d_k=128, d_v=128, states=True,
                             seed=700 + chains)
    check_against_oracle(wl, runner.backward(wl))


def test_many_short_packed_sequences():
    rng = np.random.default_rng(4242)
    lengths = [int(x) for x in rng.integers(0, 200, size=40)]
    wl = synth.make_workload("edge_many_seqs", dtype="bf16", lengths=lengths, H=3, d_k=128, d_v=128, states=True, seed=801)
    check_against_oracle(wl, runner.backward(wl))
    wl = synth.make_workload("edge_many_seqs_64", dtype="bf16", lengths=lengths, H=3, d_k=64, d_v=64, delta_rule=0,
                             g_scale=0.05, states=True, seed=802)
    check_against_oracle(wl, runner.backward(wl))
