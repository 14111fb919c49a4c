"""Host-side logic of the benchmark: workload bookkeeping and the N > 1 path (replicas with a barrier
and a max over ranks), exercised with two gloo ranks on CPU."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    # every rank times its own replica; the reported time is the slowest rank's
    mine = [10.0 + 5.0 * rank, 3.0 - rank]
    got = bench.max_over_ranks(mine, dist, "cpu")
    out[rank] = got
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_two_gloo_ranks():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1] == [15.0, 3.0]


def test_max_over_ranks_single_process_is_identity():
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]


def test_weak_scaling_value_is_sum_of_replicas():
    one = bench.aggregate_value(10**9, 1, 1.0)
    assert abs(one - 1000.0) < 1e-9
    assert abs(bench.aggregate_value(10**9, 8, 1.0) - 8 * one) < 1e-9


def test_block_spec_and_algorithmic_bytes():
    specs = [bench.block_spec(layer) for layer in range(8)]
    bits = [b for s in specs for _, b, _ in s]
    assert set(bits) == {4, 5} and len(bits) == 32
    assert len({seed for s in specs for _, _, seed in s}) == 32          # every matrix has its own seed
    from paper_2605_14844_b200 import synth
    q = synth.random_quantized(0, 64, 256, 4, 0.01, seed=3)
    want = 64 * 256 // 2 + 64 * 16 * 2 + q.nnz * 4 + 65 * 4 + 256 * 2 + 64 * 2
    assert bench.algorithmic_bytes(q) == want
    qa = synth.random_quantized(1, 64, 256, 3, 0.0, seed=3)
    assert bench.algorithmic_bytes(qa) == 64 * 256 * 3 // 8 + 32 * 8 * 2 + 64 * 2 * 5 + 65 * 4 + 256 * 2 + 64 * 2
