"""Conventions of the C ABI that the header states beside the arithmetic: calls are capturable in a CUDA graph once
the first call on the device has run, and host threads may call concurrently (each with its own stream, outputs and
workspace).  Every result is also held to the oracle's bound."""
import threading

import numpy as np
import pytest
import torch

from conftest import to_oracle
from oracle import xfp_oracle as xo
import paper_2605_14844_b200 as xfp
from paper_2605_14844_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-3


def _x_dev(x16):
    return torch.from_numpy(x16.view(np.int16)).cuda().view(torch.float16)


def _within_bound(q, x16, y):
    ref, absum = xo.gemv(to_oracle(q), x16)
    got = y.float().cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got)) and np.all(np.abs(got - ref) <= TOL * absum + 1e-30)


# shapes that reach every GEMV kernel family: batch-1 lane kernel, the kernels with two channels per lane (batch 2 on a
# small matrix), the batched lane kernel (79 row-blocks), the batched kernel with two channels per lane (8 rows), the
# general kernel (bf16 is not used here: N = 6 grouped is covered elsewhere), K slices through the workspace (96 x 12288)
CASES = [(0, 4, 200, 1024, 1), (1, 3, 200, 1024, 1), (0, 4, 200, 1024, 2), (1, 4, 200, 1024, 2), (0, 6, 2500, 768, 4),
         (1, 5, 2500, 768, 3), (0, 3, 640, 2048, 8), (1, 4, 640, 2048, 16), (0, 5, 96, 12288, 1), (1, 6, 2500, 768, 8)]


@pytest.mark.parametrize("mode,bits,rows,cols,batch", CASES)
def test_calls_are_capturable_in_a_cuda_graph(mode, bits, rows, cols, batch):
    """Three dependent-free calls captured on a side stream and replayed twice give the bits of the eager calls."""
    q = synth.random_quantized(mode, rows, cols, bits, 0.01, seed=9500 + 10 * bits + mode + batch)
    pm = xfp.pack_tensors(q, col_bits=16)
    xs = [synth.activations(batch, cols, seed=9600 + i) for i in range(3)]
    xd = [_x_dev(x) for x in xs]
    eager = [pm.gemv(x).clone() for x in xd]            # the first calls on the device: kernel attributes are set here
    torch.cuda.synchronize()
    ys = [torch.zeros_like(e) for e in eager]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for x, y in zip(xd, ys):
                pm.gemv(x, y=y, stream=side)
    for _ in range(2):
        for y in ys:
            y.zero_()
        g.replay()
        torch.cuda.synchronize()
        for e, y in zip(eager, ys):
            assert torch.equal(e, y)
    for x16, y in zip(xs, ys):
        _within_bound(q, x16, y)
    tickets = pm.workspace[: ((rows + 31) // 32) * 4].view(torch.int32)
    assert int(tickets.abs().sum().item()) == 0


def test_host_threads_call_concurrently():
    """Four host threads, each with its own stream, matrix, workspace and outputs, call the library at the same time
    (ctypes releases the interpreter lock during a call): every result equals the one the same call gave alone."""
    specs = [(0, 4, 2500, 768, 1), (1, 3, 640, 2048, 2), (0, 6, 2500, 768, 4), (1, 4, 200, 1024, 8)]
    work = []
    for i, (mode, bits, rows, cols, batch) in enumerate(specs):
        q = synth.random_quantized(mode, rows, cols, bits, 0.01, seed=9700 + i)
        pm = xfp.pack_tensors(q, col_bits=16)
        x16 = synth.activations(batch, cols, seed=9800 + i)
        xd = _x_dev(x16)
        alone = pm.gemv(xd).clone()
        torch.cuda.synchronize()
        _within_bound(q, x16, alone)
        work.append((pm, xd, alone))
    errors = []

    def run(pm, xd, alone):
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            y = torch.empty_like(alone)
            for _ in range(200):
                pm.gemv(xd, y=y, stream=stream)
            stream.synchronize()
            if not torch.equal(y, alone):
                errors.append("a concurrent call gave other bits")
        except Exception as e:  # reported on the main thread
            errors.append(repr(e))

    threads = [threading.Thread(target=run, args=w) for w in work]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
