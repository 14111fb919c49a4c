"""Single-shape driver for timing and profiling the fused GEMV.

    python -m paper_2605_14844_b200.probe launch MODE ROWS COLS BITS RATE [LAUNCHES] [PLACEMENT]
        pack one synthetic matrix and call the GEMV LAUNCHES times, evicting the matrix from L2 (a
        512 MB fill) before every call -- the target of `ncu -k regex:gemv` captures.

    python -m paper_2605_14844_b200.probe time MODE ROWS COLS BITS RATE [BATCH] [PLACEMENT] [fp16|bf16]
        time back-to-back calls over enough distinct packed copies to exceed twice the L2 (one CUDA
        graph of P calls, median of 20 replays) and print microseconds per call and effective GB/s over
        the algorithmic bytes.

    python -m paper_2605_14844_b200.probe moe [EXPERTS] [TOKENS] [BITS] [FUSED]
        routed-MoE decode layer: EXPERTS (default 128) V2a experts with a gate_up projection 3072 x 4096
        and a down projection 4096 x 1536 (one library per projection, 0.1 % outliers), top-8 routing per
        token; every token-layer is two xfp_gemv_grouped launches (8 gate_up, 8 down).  FUSED = 1 uses
        xfp_gemv_grouped_epilogue instead: SiLU(gate)*up in the store of the first launch, the routing-weighted
        sum over the experts in the store of the second (the complete expert block); FUSED = 2 computes the
        same block with the plain grouped launches and the two element-wise steps as separate kernels.
        Prints microseconds per token-layer and effective GB/s.

    python -m paper_2605_14844_b200.probe sweep [quick]
        batch and shape sweep: 8192 x 8192 and 28672 x 8192, 4-bit codebooks, V2 and V2a, x batch 1, 2, 4, 8, 16,
        outlier rate 0 / 0.3 % / 2 %, uniform and column-clustered placement (`quick`: batch 1 and 16 only).

    python -m paper_2605_14844_b200.probe stack [LAYERS]
        mixed-bit decoder stack: LAYERS (default 48) layers of q/k/v/o 4096 x 4096 plus an MLP of
        12288 x 4096 and 4096 x 12288, per-layer bit width from {2,3,4,5,6} and outlier rate from
        {0, 0.5, 1, 2} % (seeded), V2 and V2a on the same draws; one token through the stack is one CUDA graph.  Prints
        milliseconds per token and effective GB/s.

    python -m paper_2605_14844_b200.probe packdq MODE ROWS COLS BITS RATE
        device time of xfp_pack (unpacked tensors -> blob) and xfp_dequant (blob -> fp16 matrix), cold L2, with
        the bytes each must move and the resulting GB/s.

    python -m paper_2605_14844_b200.probe qkv [BITS]
        the dense-attention block (q, k, v, o 4096 x 4096, V2, ~0.9 % clustered outliers) as four calls and as
        one grouped launch for q, k, v (they share x) plus the call for o; microseconds per block.

    python -m paper_2605_14844_b200.probe quant MODE ROWS COLS BITS [REPS]
        the encoder on one synthetic float matrix (Gaussian bulk with heavy outlier columns for V2, 0.1 % uniform
        outliers for V2a): device time of every stage (statistics, extraction, Lloyd, LibFit, residual,
        cosine, median) and wall time of the whole xfp_quantize call with BITS as its only candidate.

    python -m paper_2605_14844_b200.probe gemm|gemm_v2a ROWS COLS BITS RATE M [M ...] [launch]
        the prefill form (xfp_gemm, tcgen05 tensor cores) on one V2 (gemm) or V2a (gemm_v2a, L = 32) matrix for every M given: microseconds per call
        over distinct packed copies (more than twice the L2), effective GB/s over the algorithmic bytes, TFLOP/s, and
        beside it a library fp16 GEMM (torch.matmul) on the dequantised matrix.  With `launch` as last word: three
        calls of the first M with an L2 flush before each (the target of ncu captures).

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


def time_shape(mode, rows, cols, bits, rate, batch=1, placement="uniform", reps=20, dtype="fp16"):
    from . import xfp_gemv_typed
    q = synth.random_quantized(mode, rows, cols, bits, rate, seed=1, placement=placement)
    nb = algorithmic_bytes(q, batch=batch)
    copies = max(2, int(300e6 // nb) + 1)
    pms = [pack_tensors(q, col_bits=16) for _ in range(copies)]
    x = _x(batch, cols)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float16
    if dtype == "bf16":
        x = x.to(torch.bfloat16)
    ys = [torch.empty((batch, rows), dtype=tdt, device="cuda") for _ in range(copies)]

    def call(pm, y):
        if dtype == "bf16":    # bf16 activations and outputs through the typed entry point
            xfp_gemv_typed(pm.desc, pm.packed, x, batch, y, pm.workspace)
        else:
            pm.gemv(x, y=y, y_fp16=True)

    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for pm, y in zip(pms, ys):
            call(pm, y)
        s.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            for pm, y in zip(pms, ys):
                call(pm, y)
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
    out = dict(mode=mode, rows=rows, cols=cols, bits=bits, rate=rate, batch=batch, placement=placement, dtype=dtype,
               copies=copies, MB=round(nb / 1e6, 2), us_per_call=round(t, 3), us_best=round(float(np.min(ts)), 3),
               GBs=round(nb / t / 1e3, 1))
    print(json.dumps(out), flush=True)
    return out


def moe(experts=128, tokens=64, bits=3, fused=0, distinct=8, reps=10):
    from . import XFP_EPI_COMBINE, XFP_EPI_SWIGLU, XfpDesc, xfp_gemv_grouped, xfp_gemv_grouped_epilogue, xfp_packed_size
    shapes = {"gate_up": (3072, 4096), "down": (4096, 1536)}
    packed, descs, nbytes = {}, {}, {}
    for name, (rows, cols) in shapes.items():
        base = [synth.random_quantized(1, rows, cols, bits, 0.001, seed=100 + j) for j in range(distinct)]
        for q in base[1:]:
            q.codebook = base[0].codebook            # one library per projection, shared by the layer's experts
        packed[name] = [pack_tensors(base[e % distinct], col_bits=16) for e in range(experts)]
        d0 = packed[name][0].desc
        descs[name] = XfpDesc(d0.mode, d0.rows, d0.cols, d0.bits, d0.group_size, d0.lib_size, d0.col_bits,
                              max(p.desc.nnz for p in packed[name]))
        nbytes[name] = algorithmic_bytes(base[0])
    route = synth.moe_routing(tokens, experts, 8, seed=7)
    dev = "cuda"
    x_up = [_x(1, 4096) for _ in range(tokens)]
    h = [torch.zeros((8, 1536), dtype=torch.float16, device=dev) for _ in range(tokens)]     # down inputs
    y_up = [torch.empty((8, 3072), dtype=torch.float16, device=dev) for _ in range(tokens)]
    y_dn = [torch.empty((8, 4096), dtype=torch.float16, device=dev) for _ in range(tokens)]
    y_out = [torch.empty(4096, dtype=torch.float16, device=dev) for _ in range(tokens)]
    gate_w16 = torch.full((8,), 0.125, dtype=torch.float16, device=dev)
    for t in h:
        t.copy_(_x(8, 1536))
    ptrs = lambda ts: torch.tensor([t.data_ptr() for t in ts], dtype=torch.int64, device=dev)
    args = []
    for t in range(tokens):
        ex = route[t]
        args.append((ptrs([packed["gate_up"][e].packed for e in ex]), ptrs([x_up[t]] * 8), ptrs([y_up[t][j] for j in range(8)]),
                     ptrs([packed["down"][e].packed for e in ex]), ptrs([h[t][j] for j in range(8)]),
                     ptrs([y_dn[t][j] for j in range(8)]), y_up[t], h[t], y_dn[t], y_out[t]))
    ws = {n: torch.zeros(8 * xfp_packed_size(descs[n])[1], dtype=torch.uint8, device=dev) for n in shapes}

    gate_w = torch.full((8,), 0.125, dtype=torch.float32, device=dev)   # routing weights of the token

    def layer(a):
        if fused in (3, 4):   # measurement aids: only the first (3) or only the second (4) fused store
            if fused == 3:
                xfp_gemv_grouped_epilogue(descs["gate_up"], 8, a[0], a[1], a[4], True, XFP_EPI_SWIGLU, None, ws["gate_up"])
                xfp_gemv_grouped(descs["down"], 8, a[3], a[4], a[5], True, ws["down"])
            else:
                xfp_gemv_grouped(descs["gate_up"], 8, a[0], a[1], a[2], True, ws["gate_up"])
                xfp_gemv_grouped_epilogue(descs["down"], 8, a[3], a[4], a[5], True, XFP_EPI_COMBINE, gate_w, ws["down"])
        elif fused == 1:
            # the whole expert block in two launches: gate_up with SiLU(gate)*up in its store (writes the
            # down projections' inputs), down with the routing-weighted sum over the experts in its store
            xfp_gemv_grouped_epilogue(descs["gate_up"], 8, a[0], a[1], a[4], True, XFP_EPI_SWIGLU, None, ws["gate_up"])
            xfp_gemv_grouped_epilogue(descs["down"], 8, a[3], a[4], a[5], True, XFP_EPI_COMBINE, gate_w, ws["down"])
        else:
            xfp_gemv_grouped(descs["gate_up"], 8, a[0], a[1], a[2], True, ws["gate_up"])
            if fused == 2:   # the same block with the two element-wise steps as separate (torch) kernels
                yu, hh = a[6], a[7]
                torch.mul(torch.nn.functional.silu(yu[:, :1536]), yu[:, 1536:], out=hh)
            xfp_gemv_grouped(descs["down"], 8, a[3], a[4], a[5], True, ws["down"])
            if fused == 2:
                torch.sum(a[8] * gate_w16[:, None], dim=0, out=a[9])

    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        layer(args[0])
        s.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            for a in args:
                layer(a)
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
            ts.append(e0.elapsed_time(e1) * 1e3 / tokens)
    per_layer = 8 * (nbytes["gate_up"] + nbytes["down"])
    t = float(np.median(ts))
    print(json.dumps(dict(workload=("moe_v2a", "moe_v2a_fused_ffn", "moe_v2a_ffn_with_separate_elementwise_kernels",
                                    "moe_v2a_fused_activation_only", "moe_v2a_fused_sum_only")[fused], experts=experts, tokens=tokens, bits=bits, MB_per_token_layer=round(per_layer / 1e6, 2),
                          us_per_token_layer=round(t, 2), GBs=round(per_layer / t / 1e3, 1))), flush=True)


def sweep(quick=False):
    batches = (1, 16) if quick else (1, 2, 4, 8, 16)
    for mode in (0, 1):
        for rows, cols in ((8192, 8192), (28672, 8192)):
            for rate, placement in ((0.0, "uniform"), (0.003, "uniform"), (0.003, "clustered"), (0.02, "uniform"),
                                    (0.02, "clustered")):
                for batch in batches:
                    if quick and (rate, placement) not in ((0.003, "uniform"), (0.02, "clustered")):
                        continue
                    time_shape(mode, rows, cols, 4, rate, batch, placement, reps=10)
                    torch.cuda.empty_cache()


def stack(layers=48, reps=5):
    """One token through `layers` decoder layers (6 linears each), every matrix its own packed blob."""
    shapes = [(4096, 4096)] * 4 + [(12288, 4096), (4096, 12288)]
    for mode in (0, 1):
        pms, xs, ys, total = [], {}, [], 0
        rng_l = np.random.default_rng(4)   # same bit widths and outlier rates for both modes
        cache = {}
        for layer in range(layers):
            bits = int(rng_l.integers(2, 7))
            rate = (0.0, 0.005, 0.01, 0.02)[int(rng_l.integers(0, 4))]
            for j, (rows, cols) in enumerate(shapes):
                # layers that drew the same (bits, rate) reuse the host tensors; every layer packs its own blobs
                key = (bits, rate, j)
                if key not in cache:
                    cache[key] = synth.random_quantized(mode, rows, cols, bits, rate, seed=5000 + 97 * len(cache) + j)
                q = cache[key]
                pms.append(pack_tensors(q, col_bits=16))
                total += algorithmic_bytes(q)
                xs.setdefault(cols, _x(1, cols))
                ys.append(torch.empty((1, rows), dtype=torch.float16, device="cuda"))
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            def token():
                for pm, y in zip(pms, ys):
                    pm.gemv(xs[pm.desc.cols], y=y, y_fp16=True)
            token()
            s.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                token()
            for _ in range(2):
                g.replay()
            s.synchronize()
            ts = []
            for _ in range(reps):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(s)
                g.replay()
                e1.record(s)
                s.synchronize()
                ts.append(e0.elapsed_time(e1))
        t = float(np.median(ts))
        print(json.dumps(dict(workload="decoder_stack", mode=mode, layers=layers, calls=len(pms), GB_per_token=round(total / 1e9, 3),
                              ms_per_token=round(t, 4), GBs=round(total / t / 1e6, 1))), flush=True)
        del pms, ys
        torch.cuda.empty_cache()


def packdq(mode, rows, cols, bits, rate, reps=10):
    """Device time of xfp_pack and xfp_dequant on one matrix, with the bytes each has to move."""
    from . import XfpDesc, xfp_dequant, xfp_pack, xfp_packed_size
    from .binding import _dev
    q = synth.random_quantized(mode, rows, cols, bits, rate, seed=1)
    nnz = int(q.rowptr[-1])
    desc = XfpDesc(q.mode, q.rows, q.cols, q.bits, q.group_size, q.lib_size if q.mode else 0, 16, nnz)
    pb, _ = xfp_packed_size(desc)
    dev = "cuda"
    idx, cb = _dev(q.idx, torch.uint8, dev), _dev(q.codebook, torch.int16, dev)
    gid = _dev(q.gid, torch.uint8, dev) if mode else None
    gs = _dev(q.gscale, torch.int16, dev) if mode else None
    gm = _dev(q.gmid, torch.int16, dev) if mode else None
    rowptr = _dev(q.rowptr, torch.int32, dev)
    ocol = _dev(q.ocol.astype(np.uint16), torch.int16, dev)
    oval = _dev(q.oval, torch.int16, dev)
    packed = torch.empty(pb, dtype=torch.uint8, device=dev)
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    Wout = torch.empty((rows, cols), dtype=torch.float16, device=dev)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)

    def timed(fn):
        ts = []
        for _ in range(reps + 2):
            flush.fill_(1)     # inputs and outputs start outside L2
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3)
        return float(np.median(ts[2:]))

    t_pack = timed(lambda: xfp_pack(desc, idx, cb, gid, gs, gm, rowptr, ocol, oval, packed, err))
    t_dq = timed(lambda: xfp_dequant(desc, packed, Wout))
    meta = algorithmic_bytes(q) - rows * cols * bits // 8
    pack_bytes = rows * cols + rows * cols * bits // 8 + 2 * meta       # byte indices in, bit stream out, metadata in and out
    dq_bytes = rows * cols * bits // 8 + meta + rows * cols * 2          # blob in, fp16 matrix out
    print(json.dumps(dict(workload="pack_dequant", mode=mode, rows=rows, cols=cols, bits=bits, rate=rate, nnz=nnz,
                          pack_us=round(t_pack, 1), pack_MB=round(pack_bytes / 1e6, 1), pack_GBs=round(pack_bytes / t_pack / 1e3, 1),
                          dequant_us=round(t_dq, 1), dequant_MB=round(dq_bytes / 1e6, 1),
                          dequant_GBs=round(dq_bytes / t_dq / 1e3, 1), err_word=int(err.item()))), flush=True)


def qkv(bits=4, reps=20):
    """The attention block's q, k, v (shared x) as three calls against one grouped launch; o stays a call of its own."""
    from . import XfpDesc, xfp_gemv_grouped, xfp_packed_size
    rows = cols = 4096
    sets = max(2, int(300e6 // (4 * rows * cols * bits // 8)) + 1)
    blocks = []
    nb = 0
    for st in range(sets):
        qs = [synth.random_quantized(0, rows, cols, bits, 0.009, seed=10 + j, placement="clustered") for j in range(4)]
        blocks.append([pack_tensors(q, col_bits=16) for q in qs])
        nb = sum(algorithmic_bytes(q) for q in qs)
    x = _x(1, cols)
    ys = [torch.empty((4, rows), dtype=torch.float16, device="cuda") for _ in range(sets)]
    d0 = blocks[0][0].desc
    desc = XfpDesc(d0.mode, d0.rows, d0.cols, d0.bits, d0.group_size, d0.lib_size, d0.col_bits,
                   max(p.desc.nnz for b in blocks for p in b))
    ws = torch.zeros(3 * xfp_packed_size(desc)[1], dtype=torch.uint8, device="cuda")
    ptrs = lambda ts: torch.tensor([t.data_ptr() for t in ts], dtype=torch.int64, device="cuda")
    lists = [(ptrs([p.packed for p in b[:3]]), ptrs([x] * 3), ptrs([y[j] for j in range(3)])) for b, y in zip(blocks, ys)]
    out = {}
    for name in ("four_calls", "grouped_qkv_plus_o"):
        def block(i):
            b, y = blocks[i], ys[i]
            if name == "four_calls":
                for j in range(3):
                    b[j].gemv(x, y=y[j:j + 1], y_fp16=True)
            else:
                xfp_gemv_grouped(desc, 3, lists[i][0], lists[i][1], lists[i][2], True, ws)
            b[3].gemv(x, y=y[3:4], y_fp16=True)
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            for i in range(sets):
                block(i)
            s.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                for i in range(sets):
                    block(i)
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
                ts.append(e0.elapsed_time(e1) * 1e3 / sets)
        out[name + "_us_per_block"] = round(float(np.median(ts)), 3)
        out[name + "_GBs"] = round(nb / float(np.median(ts)) / 1e3, 1)
    print(json.dumps(dict(workload="attention_block_qkv_o", bits=bits, MB_per_block=round(nb / 1e6, 2), **out)), flush=True)


def quant(mode, rows, cols, bits, reps=3):
    """Device time per encoder stage, and the whole Algorithm 1 call, on one rows x cols float matrix."""
    from . import XfpDesc
    from . import quant_binding as qb
    if mode == 0:
        W = synth.attention_weights(10, rows, cols)
    else:
        W = synth.plant_uniform_outliers(synth.gaussian_weights(rows, cols, 30), 0.001, 31)
    Wd = torch.from_numpy(W).cuda()
    L = 32
    cap = int(0.02 * W.size)
    buf = qb.QuantBuffers(rows, cols, mode, bits, L, cap)
    ms = torch.zeros(2, dtype=torch.float64, device="cuda")
    cnt = torch.zeros(2, dtype=torch.int64, device="cuda")
    med = torch.zeros(2, dtype=torch.float64, device="cuda")
    desc = XfpDesc(mode, rows, cols, bits, 128, L if mode else 0, 32, 0)
    table = buf.lib if mode else buf.codebook
    stages = [
        ("stats", lambda: qb.xfp_quant_stats(Wd, 0, ms, buf.workspace)),
        ("outliers", lambda: qb.xfp_quant_outliers(Wd, ms, 0, 4.0, 0.02, buf.mask, cnt, buf.workspace)),
        ("lloyd", lambda: qb.xfp_quant_lloyd(Wd, buf.mask, ms, bits, 20, buf.codebook, buf.idx, buf.workspace)),
    ]
    if mode:
        stages += [
            ("libfit_library", lambda: qb.xfp_quant_libfit_library(buf.codebook, rows, bits, L, 20, buf.lib, buf.workspace)),
            ("libfit_assign", lambda: qb.xfp_quant_libfit_assign(Wd, buf.mask, ms, bits, L, buf.lib, buf.idx, buf.gid,
                                                                 buf.gscale, buf.gmid)),
        ]
    stages += [
        ("residual", lambda: qb.xfp_quant_residual(desc, Wd, buf.mask, buf.idx, table, buf.gid, buf.gscale, buf.gmid,
                                                   buf.rowptr, buf.ocol, buf.oval, buf.workspace)),
        ("cosine", lambda: qb.xfp_quant_cosine(desc, Wd, buf.mask, buf.idx, table, buf.gid, buf.gscale, buf.gmid, buf.cos)),
        ("median", lambda: qb.xfp_quant_median(buf.cos, med, buf.workspace)),
    ]
    out = {}
    for name, fn in stages:
        fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        out[name + "_ms"] = round(float(np.median(ts)), 4)
    import time
    params = qb.XfpQuantParams(0, 0, 4.0, 0.02, 0.0, 20, 0)
    walls = []
    for _ in range(reps):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        res = qb.xfp_quantize(mode, Wd, params, (bits,), 0.0, buf)
        torch.cuda.synchronize()
        walls.append((time.perf_counter() - t0) * 1e3)
    print(json.dumps(dict(workload="encoder", mode=mode, rows=rows, cols=cols, bits=bits, nnz=int(res.nnz),
                          median_cos=round(res.median_cos, 6), stages=out, stage_sum_ms=round(sum(out.values()), 3),
                          quantize_wall_ms=round(float(np.median(walls)), 3),
                          Mweights_per_s=round(rows * cols / np.median(walls) / 1e3, 1))), flush=True)


def gemm(rows, cols, bits, rate, ms, launch_only=False, reps=20, mode=0):
    from . import xfp_gemm, xfp_gemm_workspace_size
    q = synth.random_quantized(mode, rows, cols, bits, rate, seed=1)
    if launch_only:
        pm = pack_tensors(q, col_bits=16)
        m = ms[0]
        x = _x(m, cols)
        y = torch.empty((m, rows), dtype=torch.float16, device="cuda")
        ws = torch.zeros(xfp_gemm_workspace_size(pm.desc, m), dtype=torch.uint8, device="cuda")
        flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
        for _ in range(3):
            flush.fill_(1)
            xfp_gemm(pm.desc, pm.packed, x, y, ws)
        torch.cuda.synchronize()
        print("ok", float(y.float().abs().sum()), int(ws[:4].view(torch.int32).item()))
        return
    nb0 = algorithmic_bytes(q, batch=0)
    copies = max(2, int(300e6 // nb0) + 1)
    pms = [pack_tensors(q, col_bits=16) for _ in range(copies)]
    W = pms[0].dequant()
    s = torch.cuda.Stream()

    def timed(fn):
        with torch.cuda.stream(s):
            fn()
            s.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                fn()
            # replay for half a second first: the SM clock needs tens of milliseconds of load to leave its idle state
            import time
            t_end = time.time() + 0.5
            while time.time() < t_end:
                for _ in range(10):
                    g.replay()
                s.synchronize()
            ts = []
            for _ in range(reps):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(s)
                g.replay()
                e1.record(s)
                s.synchronize()
                ts.append(e0.elapsed_time(e1) * 1e3)
        return float(np.median(ts))

    for m in ms:
        x = _x(m, cols)
        ys = [torch.empty((m, rows), dtype=torch.float16, device="cuda") for _ in range(copies)]
        wss = [torch.zeros(xfp_gemm_workspace_size(pm.desc, m), dtype=torch.uint8, device="cuda") for pm in pms]
        t = timed(lambda: [xfp_gemm(pm.desc, pm.packed, x, y, ws) for pm, y, ws in zip(pms, ys, wss)]) / copies
        Ws = [W.clone() for _ in range(max(2, int(300e6 // (rows * cols * 2)) + 1))]
        t_lib = timed(lambda: [torch.matmul(x, w.t(), out=ys[0]) for w in Ws]) / len(Ws)
        nb = nb0 + m * (cols * 2 + rows * 2)
        fl = 2.0 * m * rows * cols
        err = max(int(ws[:4].view(torch.int32).item()) for ws in wss)
        print(json.dumps(dict(mode=mode, rows=rows, cols=cols, bits=bits, rate=rate, M=m, copies=copies, us_per_call=round(t, 2),
                              GBs=round(nb / t / 1e3, 1), TFLOPs=round(fl / t / 1e6, 1),
                              lib_fp16_gemm_us=round(t_lib, 2), err_flag=err)), flush=True)


def main(argv):
    if len(argv) > 1 and argv[1] in ("gemm", "gemm_v2a"):
        lo = argv[-1] == "launch"
        rest = argv[6:-1] if lo else argv[6:]
        gemm(int(argv[2]), int(argv[3]), int(argv[4]), float(argv[5]), [int(v) for v in rest], lo,
             mode=1 if argv[1] == "gemm_v2a" else 0)
        return 0
    if len(argv) > 1 and argv[1] == "packdq":
        packdq(int(argv[2]), int(argv[3]), int(argv[4]), int(argv[5]), float(argv[6]))
        return 0
    if len(argv) > 1 and argv[1] == "qkv":
        qkv(*(int(v) for v in argv[2:3]))
        return 0
    if len(argv) > 1 and argv[1] == "quant":
        quant(*(int(v) for v in argv[2:7]))
        return 0
    if len(argv) > 1 and argv[1] == "moe":
        moe(*(int(v) for v in argv[2:6]))
        return 0
    if len(argv) > 1 and argv[1] == "sweep":
        sweep(len(argv) > 2 and argv[2] == "quick")
        return 0
    if len(argv) > 1 and argv[1] == "stack":
        stack(*(int(v) for v in argv[2:3]))
        return 0
    if len(argv) < 7 or argv[1] not in ("launch", "time"):
        print(__doc__)
        return 2
    mode, rows, cols, bits = (int(v) for v in argv[2:6])
    rate = float(argv[6])
    if argv[1] == "launch":
        launch(mode, rows, cols, bits, rate, int(argv[7]) if len(argv) > 7 else 3, argv[8] if len(argv) > 8 else "uniform")
    else:
        time_shape(mode, rows, cols, bits, rate, int(argv[7]) if len(argv) > 7 else 1,
                   argv[8] if len(argv) > 8 else "uniform", dtype=argv[9] if len(argv) > 9 else "fp16")
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv))
