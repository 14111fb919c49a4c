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


def test_stack_spec_matches_the_configuration():
    """The headline workload's per-layer draws: 48 layers, bit widths from {2..6}, outlier rates within [0, 2 %]."""
    from paper_2605_14844_b200 import workloads as wl
    spec = wl.stack_spec()
    assert len(spec) == 48 and spec == wl.stack_spec()                    # seeded
    assert {b for b, _ in spec} == {2, 3, 4, 5, 6}
    assert all(0.0 <= r <= 0.02 for _, r in spec)
    assert wl.STACK_SHAPES == [(4096, 4096)] * 4 + [(12288, 4096), (4096, 12288)]
    total = sum(wl.algorithmic_bytes(0, r, c, b, int(rate * r * c)) for b, rate in spec for r, c in wl.STACK_SHAPES)
    assert 3.5e9 < total < 5.5e9                                          # about 4.4 GB per token


def test_device_generator_follows_the_host_recipe():
    """synth.random_quantized_torch (here on the CPU device) gives tensors of the recipe's shapes, ranges and
    structure; to_host returns them in the oracle's types."""
    from paper_2605_14844_b200 import synth
    for mode in (0, 1):
        for placement in ("uniform", "clustered"):
            q = synth.to_host(synth.random_quantized_torch(mode, 96, 512, 3, 0.01, 5, placement, device="cpu"))
            assert q.idx.shape == (96, 512) and q.idx.dtype == np.uint8 and q.idx.max() <= 7
            assert q.rowptr[0] == 0 and q.rowptr[-1] == q.ocol.size == q.oval.size
            assert 0.5 * 0.01 * 96 * 512 < q.nnz < 1.5 * 0.01 * 96 * 512
            for i in range(96):
                c = q.ocol[q.rowptr[i]:q.rowptr[i + 1]]
                assert np.all(np.diff(c) > 0) and (c.size == 0 or (0 <= c[0] and c[-1] < 512))
            cb = q.codebook.view(np.float16).astype(np.float64)
            assert np.all(np.diff(cb, axis=1) >= 0)
            mag = np.abs(q.oval.view(np.float16).astype(np.float64))
            assert np.all((mag >= 0.199) & (mag <= 0.981))                # 10..49 sigma
            if mode:
                assert q.gid.shape == (96, 4) and q.gid.max() < 32 and q.codebook.shape == (32, 8)
