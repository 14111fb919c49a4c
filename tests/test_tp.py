"""Tensor-parallel row split ("Setup": the paper deploys at TP = 2): partition arithmetic and shard contents on the
host, the all-gather with two gloo ranks on CPU (the oracle computes each rank's slice), and on the GPU the shards of
a two-way split run one after the other on one device."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from conftest import to_oracle
from oracle import xfp_oracle as xo
from paper_2605_14844_b200 import synth, tp


def test_row_partition_tiles_the_rows_at_row_block_boundaries():
    for rows in (1, 31, 32, 33, 70, 4096, 4097, 28672):
        for world in (1, 2, 3, 4, 8):
            per, parts = tp.row_partition(rows, world)
            assert per % 32 == 0 and len(parts) == world
            assert parts[0][0] == 0 and parts[-1][1] == rows
            for (a0, a1), (b0, b1) in zip(parts, parts[1:]):
                assert a1 == b0 and a0 <= a1
            assert all(r0 % 32 == 0 for r0, _ in parts if r0 < rows)
            assert all(r1 - r0 <= per for r0, r1 in parts)
            assert per * world >= rows and per * (world - 1) < rows + 32 * world


@pytest.mark.parametrize("mode", [0, 1])
def test_shards_hold_exactly_their_rows(mode):
    q = synth.random_quantized(mode, 70, 256, 3, 0.03, seed=91 + mode)
    full = xo.dequant(to_oracle(q))
    got = []
    for r in range(2):
        s = tp.shard_tensors(q, r, 2)
        assert s.rowptr[0] == 0 and s.rowptr[-1] == s.ocol.size == s.oval.size
        got.append(xo.dequant(to_oracle(s)))
    assert np.array_equal(np.concatenate(got, axis=0), full)
    assert tp.shard_tensors(synth.random_quantized(0, 20, 128, 2, 0.0, seed=1), 1, 2) is None   # a rank without rows


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    q = synth.random_quantized(1, 200, 512, 4, 0.01, seed=92)
    x16 = synth.activations(2, 512, seed=93)
    per, parts = tp.row_partition(q.rows, world)
    shard = tp.shard_tensors(q, rank, world)
    local = np.zeros((2, per))
    y, _ = xo.gemv(to_oracle(shard), x16)             # this rank's rows, by the oracle
    local[:, :y.shape[1]] = y
    out[rank] = tp.gather_rows(local, q.rows, world, dist)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_gather_the_full_result():
    world = 2
    port = 29600 + (os.getpid() % 2000)
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        q = synth.random_quantized(1, 200, 512, 4, 0.01, seed=92)
        ref, _ = xo.gemv(to_oracle(q), synth.activations(2, 512, seed=93))
        assert np.array_equal(out[0], ref) and np.array_equal(out[1], ref)   # rows are independent: identical bits


@pytest.mark.gpu
@pytest.mark.parametrize("mode,bits", [(0, 4), (1, 3)])
def test_shards_on_the_gpu_reproduce_the_layer(mode, bits):
    import paper_2605_14844_b200 as xfp
    q = synth.random_quantized(mode, 1000, 1024, bits, 0.01, seed=94 + mode)
    x16 = synth.activations(1, 1024, seed=95)
    x = torch.from_numpy(x16.view(np.int16)).cuda().view(torch.float16)
    ref, absum = xo.gemv(to_oracle(q), x16)
    per, parts = tp.row_partition(q.rows, 2)
    got = np.zeros((1, 2 * per))
    for r in range(2):                                   # the two ranks' launches, one after the other on this GPU
        pm = xfp.pack_tensors(tp.shard_tensors(q, r, 2), col_bits=16)
        y = pm.gemv(x)
        torch.cuda.synchronize()
        got[:, r * per:r * per + y.shape[1]] = y.cpu().numpy()
    assert np.all(np.abs(got[:, :q.rows] - ref) <= 1e-3 * absum + 1e-30)
    # the single-process form of the layer object (world size 1) gives the whole y
    layer = tp.TpLinear(q, "cuda")
    y1 = layer.gemv(x, y_fp16=False)
    torch.cuda.synchronize()
    assert y1.shape == (1, q.rows)
    assert np.all(np.abs(y1.cpu().numpy().astype(np.float64) - ref) <= 1e-3 * absum + 1e-30)
