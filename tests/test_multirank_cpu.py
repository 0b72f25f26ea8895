"""The N > 1 path of the benchmark on CPU: two gloo ranks, independent batches, no data-path collective.
Only the timing protocol communicates (max elapsed time over ranks, total units over ranks)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_12700_b200 import benchutil, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # every rank owns its own batch of the same shape: heads permuted per rank as bench.py does
        wl = synth.make_workload("rank_batch", dtype="bf16", B=1, T=128, H=4, d_k=64, d_v=64, seed=3)
        elapsed_ms = 10.0 + 5.0 * rank            # rank 1 is the slow one
        t, u = benchutil.aggregate_over_ranks(elapsed_ms, wl.tokens * 7, dist, torch.device("cpu"))
        dist.barrier()
        out[rank] = (t, u)
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_the_max_time_and_sum_the_tokens():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert out[0] == out[1] == (15.0, 2.0 * 128 * 7)
    # whole-job throughput = units of all ranks / slowest rank's time
    t, u = out[0]
    assert abs(u / (t * 1e-3) - 2 * 128 * 7 / 15e-3) < 1e-6


def test_single_process_is_a_no_op():
    assert benchutil.aggregate_over_ranks(3.5, 100.0, None, None) == (3.5, 100.0)


def test_roofline_bookkeeping_matches_hand_counts():
    # cfg1: 131072 token-heads, 64 chains, 2048 chunk-heads, bf16, d = 128, states present
    b = benchutil.path_alg_bytes(token_heads=131072, chains=64, d_k=128, d_v=128, io_bytes=2, delta_rule=1,
                                 has_h0=True, has_dhT=True)
    assert b == 131072 * 1808 + 64 * 3 * 128 * 128 * 4
    f = benchutil.path_alg_flops(chunk_heads=2048, d_k=128, d_v=128, delta_rule=1)
    assert abs(f / 2048 - (14 * 64 * 64 * 128 + 8 * 2 * 64 * 128 * 128 + 2 * 64 ** 3 / 3)) < 1
    # cfg2: d = 64, delta rule off: 904 B per token-head
    assert benchutil.path_alg_bytes(token_heads=1, chains=0, d_k=64, d_v=64, io_bytes=2, delta_rule=0,
                                    has_h0=False, has_dhT=False) == 904
