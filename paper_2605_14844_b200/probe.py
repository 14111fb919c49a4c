"""Single-shape driver for timing and profiling the fused GEMV.

    python -m paper_2605_14844_b200.probe launch MODE ROWS COLS BITS RATE [LAUNCHES] [PLACEMENT]
        pack one synthetic matrix and call the GEMV LAUNCHES times, evicting the matrix from L2 (a
        512 MB fill) before every call -- the target of `ncu -k regex:gemv` captures.

    python -m paper_2605_14844_b200.probe time MODE ROWS COLS BITS RATE [BATCH] [PLACEMENT]
        time back-to-back calls over enough distinct packed copies to exceed twice the L2 (one CUDA
        graph of P calls, median of 20 replays) and print microseconds per call and effective GB/s over
        the algorithmic bytes.

MODE 0 = V2, 1 = V2a; PLACEMENT uniform | clustered | one_row.  Inputs come from synth.random_quantized.
"""
from __future__ import annotations

import json
import sys

import numpy as np
import torch

from . import pack_tensors, synth


def algorithmic_bytes(q, y_bytes: int = 2, batch: int = 1) -> int:
    """Bytes the method must move for one call: indices, codebooks / library and group metadata,
    outlier values and columns, row pointers, x and y."""
    E = 1 << q.bits
    b = q.rows * q.cols * q.bits // 8 + (q.rows if q.mode == 0 else q.lib_size) * E * 2
    if q.mode:
        b += q.rows * (q.cols // q.group_size) * 5
    return b + q.nnz * 4 + (q.rows + 1) * 4 + batch * (q.cols * 2 + q.rows * y_bytes)


def _x(batch, cols):
    return torch.from_numpy(synth.activations(batch, cols, 3).view(np.int16)).cuda().view(torch.float16)


def launch(mode, rows, cols, bits, rate, n=3, placement="uniform"):
    q = synth.random_quantized(mode, rows, cols, bits, rate, seed=1, placement=placement)
    pm = pack_tensors(q, col_bits=16)
    x = _x(1, cols)
    y = torch.empty((1, rows), dtype=torch.float16, device="cuda")
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    for _ in range(n):
        flush.fill_(1)
        pm.gemv(x, y=y, y_fp16=True)
    torch.cuda.synchronize()
    print("ok", float(y.float().abs().sum()))


def time_shape(mode, rows, cols, bits, rate, batch=1, placement="uniform", reps=20):
    q = synth.random_quantized(mode, rows, cols, bits, rate, seed=1, placement=placement)
    nb = algorithmic_bytes(q, batch=batch)
    copies = max(2, int(300e6 // nb) + 1)
    pms = [pack_tensors(q, col_bits=16) for _ in range(copies)]
    x = _x(batch, cols)
    ys = [torch.empty((batch, rows), dtype=torch.float16, device="cuda") for _ in range(copies)]
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for pm, y in zip(pms, ys):
            pm.gemv(x, y=y, y_fp16=True)
        s.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            for pm, y in zip(pms, ys):
                pm.gemv(x, y=y, y_fp16=True)
        for _ in range(3):
            g.replay()
        s.synchronize()
        ts = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(s)
            g.replay()
            e1.record(s)
            s.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3 / copies)
    t = float(np.median(ts))
    out = dict(mode=mode, rows=rows, cols=cols, bits=bits, rate=rate, batch=batch, placement=placement,
               copies=copies, MB=round(nb / 1e6, 2), us_per_call=round(t, 3), us_best=round(float(np.min(ts)), 3),
               GBs=round(nb / t / 1e3, 1))
    print(json.dumps(out), flush=True)
    return out


def main(argv):
    if len(argv) < 7 or argv[1] not in ("launch", "time"):
        print(__doc__)
        return 2
    mode, rows, cols, bits = (int(v) for v in argv[2:6])
    rate = float(argv[6])
    if argv[1] == "launch":
        launch(mode, rows, cols, bits, rate, int(argv[7]) if len(argv) > 7 else 3, argv[8] if len(argv) > 8 else "uniform")
    else:
        time_shape(mode, rows, cols, bits, rate, int(argv[7]) if len(argv) > 7 else 1,
                   argv[8] if len(argv) > 8 else "uniform")
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv))
