"""Synthetic workloads shaped like the paper's layers, prepared on the device and timed as CUDA graphs.

Each workload is a list of fused-GEMV calls over packed blobs (drawn by synth.random_quantized_torch, packed by
xfp_pack) plus the algorithmic bytes one pass over them must move: packed indices, codebooks or library and group
metadata, outlier values and columns, row pointers, x and y ("Fused Decode Kernel"; bytes as in the format
section's storage accounting, with 4 bytes per outlier).  `bench.py` times them; the same objects serve as small,
single-kernel targets for profiler captures (`bench.py --workload NAME --launches N`).

    stack         48 decoder layers x (q, k, v, o 4096 x 4096, 12288 x 4096, 4096 x 12288), per-layer bit width from
                  {2..6} and outlier rate from [0, 2 %] (seeded), V2 or V2a on the same draws; one token = 288 calls
    attention     blocks of q/k/v/o 4096 x 4096, V2, N from {4, 5}, ~0.9 % outliers in heavy outlier columns
                  (attention_grouped: q, k and v of a block in one grouped launch)
    single        one 4096 x 4096 V2 layer, N = 4, 0.3 % uniform outliers, cycled over distinct copies
    moe           routed-MoE token-layers: 128 experts (gate_up 3072 x 4096, down 4096 x 1536), V2a N = 3, L = 32,
                  0.1 % outliers, top-8 routing; a token-layer is two grouped launches with fused stores
    shape         one matrix of any shape / mode / bits / outlier rate / batch, cycled over distinct copies
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Callable, List, Optional

import numpy as np
import torch

from . import binding as xb
from . import synth

L2_BYTES = 126 << 20


def algorithmic_bytes(mode: int, rows: int, cols: int, bits: int, nnz: int, lib_size: int = 32, group_size: int = 128,
                      batch: int = 1, y_bytes: int = 2) -> int:
    """Bytes one fused GEMV call must move."""
    E = 1 << bits
    b = rows * cols * bits // 8 + (rows if mode == 0 else lib_size) * E * 2
    if mode:
        b += rows * (cols // group_size) * 5          # id u8 + scale fp16 + mid fp16 per group
    return b + nnz * 4 + (rows + 1) * 4 + batch * (cols * 2 + rows * y_bytes)


@dataclass
class Workload:
    name: str
    config: dict
    run: Callable[[], None]              # queue one step on the current stream
    bytes_per_step: int
    calls_per_step: int                  # fused GEMV calls (a grouped launch over n blobs counts n)
    launches_per_step: int               # kernels of this library launched per step
    keep: list = field(default_factory=list)      # device tensors that must stay alive
    host_step: Optional[Callable] = None          # the same step through xfp_gemv_host (pinned host x in, y out)
    h2d_bytes: int = 0
    d2h_bytes: int = 0
    sample: list = field(default_factory=list)    # a few (QuantTensors on the device, x16 numpy) for the CPU oracle


def _x(batch: int, cols: int, seed: int, device) -> torch.Tensor:
    return torch.from_numpy(synth.activations(batch, cols, seed).view(np.int16)).to(device).view(torch.float16)


def _pack(q, device):
    pm = xb.pack_tensors(q, device=device, col_bits=16)
    return pm


def _bytes_of(pm, batch=1, y_bytes=2) -> int:
    d = pm.desc
    return algorithmic_bytes(d.mode, d.rows, d.cols, d.bits, d.nnz, d.lib_size, d.group_size, batch, y_bytes)


STACK_SHAPES = [(4096, 4096)] * 4 + [(12288, 4096), (4096, 12288)]


def stack_spec(layers: int = 48, seed: int = 4):
    """(bits, outlier rate) per layer: N uniform on {2..6}, rate uniform on [0, 2 %] in steps of 0.1 %."""
    rng = np.random.default_rng(seed)
    return [(int(rng.integers(2, 7)), float(rng.integers(0, 21)) / 1000.0) for _ in range(layers)]


def stack(mode: int, layers: int = 48, device="cuda", with_host: bool = False, n_sample: int = 0) -> Workload:
    spec = stack_spec(layers)
    pms, xs, ys, total, sample = [], {}, [], 0, []
    for li, (bits, rate) in enumerate(spec):
        for j, (rows, cols) in enumerate(STACK_SHAPES):
            q = synth.random_quantized_torch(mode, rows, cols, bits, rate, seed=5000 + 16 * li + j, device=device)
            pm = _pack(q, device)
            if len(sample) < n_sample:
                sample.append((synth.to_host(q), synth.activations(1, cols, 900 + cols)))
            del q
            pms.append(pm)
            total += _bytes_of(pm)
            if cols not in xs:
                xs[cols] = _x(1, cols, 900 + cols, device)
            ys.append(torch.empty((1, rows), dtype=torch.float16, device=device))
    torch.cuda.synchronize(device)
    assert all(int(p.err_word.item()) == 0 for p in pms)

    def run():
        for pm, y in zip(pms, ys):
            pm.gemv(xs[pm.desc.cols], y=y, y_fp16=True)

    w = Workload("stack_v2a" if mode else "stack_v2",
                 {"workload": "48-layer mixed-bit decoder linear sweep (configuration 4)" if layers == 48 else
                  f"{layers}-layer mixed-bit decoder linear sweep", "mode": "V2a" if mode else "V2", "layers": layers,
                  "linears_per_layer": "q,k,v,o 4096x4096 + 12288x4096 + 4096x12288", "batch": 1,
                  "bits_per_layer": [s[0] for s in spec], "outlier_rate_per_layer": [s[1] for s in spec],
                  "x": "fp16", "y": "fp16"},
                 run, total, len(pms), len(pms), keep=[pms, xs, ys], sample=sample)
    if with_host:
        xh = {c: torch.from_numpy(synth.activations(1, c, 900 + c).view(np.int16)).pin_memory() for c in xs}
        xstage = [torch.empty((1, pm.desc.cols), dtype=torch.float16, device=device) for pm in pms]
        yh = [torch.empty((1, pm.desc.rows), dtype=torch.float16).pin_memory() for pm in pms]

        def host_step(stream):
            for pm, xd, yhost, yd in zip(pms, xstage, yh, ys):
                xb.xfp_gemv_host(pm.desc, pm.packed, xh[pm.desc.cols], xd, 1, yhost, yd, True, pm.workspace, stream)

        w.host_step = host_step
        w.h2d_bytes = sum(pm.desc.cols * 2 for pm in pms)
        w.d2h_bytes = sum(pm.desc.rows * 2 for pm in pms)
        w.keep += [xh, xstage, yh]
    return w


def attention(layers: int = 8, device="cuda") -> Workload:
    pms, ys, total, bits_used = [], [], 0, []
    for layer in range(layers):
        rng = np.random.default_rng(1000 + layer)
        for j, b in enumerate(rng.integers(4, 6, size=4)):
            q = synth.random_quantized_torch(0, 4096, 4096, int(b), 0.009, seed=10 + 4 * layer + j,
                                             placement="clustered", device=device)
            pms.append(_pack(q, device))
            total += _bytes_of(pms[-1])
            bits_used.append(int(b))
            ys.append(torch.empty((1, 4096), dtype=torch.float16, device=device))
    x = _x(1, 4096, 900, device)

    def run():
        for pm, y in zip(pms, ys):
            pm.gemv(x, y=y, y_fp16=True)

    return Workload("attention", {"workload": "dense attention blocks (configuration 2)", "mode": "V2", "blocks": layers,
                                  "projections": "q,k,v,o 4096x4096", "bits": bits_used[:4], "outlier_rate": 0.009,
                                  "placement": "heavy outlier columns", "batch": 1},
                    run, total, len(pms), len(pms), keep=[pms, ys, x])


def attention_grouped(layers: int = 8, device="cuda") -> Workload:
    """The same blocks with q, k and v (they share x) in one grouped launch per block and o as a call of its own;
    a block's q/k/v take one bit width (a grouped launch has one descriptor)."""
    blocks, total, bits_used, keep = [], 0, [], []
    x = _x(1, 4096, 900, device)
    ptrs = lambda ts: torch.tensor([t.data_ptr() for t in ts], dtype=torch.int64, device=device)
    for layer in range(layers):
        rng = np.random.default_rng(1000 + layer)
        b_qkv, b_o = (int(v) for v in rng.integers(4, 6, size=2))
        pms = [_pack(synth.random_quantized_torch(0, 4096, 4096, b_qkv if j < 3 else b_o, 0.009, seed=10 + 4 * layer + j,
                                                  placement="clustered", device=device), device) for j in range(4)]
        total += sum(_bytes_of(pm) for pm in pms)
        bits_used += [b_qkv] * 3 + [b_o]
        y = torch.empty((4, 4096), dtype=torch.float16, device=device)
        d0 = pms[0].desc
        desc = xb.XfpDesc(d0.mode, d0.rows, d0.cols, d0.bits, d0.group_size, d0.lib_size, d0.col_bits,
                          max(p.desc.nnz for p in pms[:3]))
        ws = torch.zeros(3 * xb.xfp_packed_size(desc)[1], dtype=torch.uint8, device=device)
        blocks.append((desc, ptrs([p.packed for p in pms[:3]]), ptrs([x] * 3), ptrs([y[j] for j in range(3)]), ws, pms[3], y))
        keep.append(pms)

    def run():
        for desc, pp, px, py, ws, po, y in blocks:
            xb.xfp_gemv_grouped(desc, 3, pp, px, py, True, ws)
            po.gemv(x, y=y[3:4], y_fp16=True)

    return Workload("attention_grouped", {"workload": "dense attention blocks, q/k/v in one grouped launch", "mode": "V2",
                                          "blocks": layers, "bits": bits_used[:4], "outlier_rate": 0.009, "batch": 1},
                    run, total, 4 * layers, 2 * layers, keep=[blocks, keep, x])


def shape(mode: int, rows: int, cols: int, bits: int, rate: float, batch: int = 1, placement: str = "uniform",
          device="cuda", name: Optional[str] = None, copies: Optional[int] = None, seed: int = 1) -> Workload:
    """One matrix cycled over enough distinct packed copies to exceed twice the L2."""
    q = synth.random_quantized_torch(mode, rows, cols, bits, rate, seed=seed, placement=placement, device=device)
    first = _pack(q, device)
    nb = _bytes_of(first, batch)
    if copies is None:
        copies = max(2, int(2 * L2_BYTES // nb) + 1)
    pms = [first]
    for _ in range(copies - 1):
        pm = xb.PackedMatrix(first.desc, first.packed.clone(), torch.zeros_like(first.workspace), first.err_word)
        pms.append(pm)
    x = _x(batch, cols, 3, device)
    ys = [torch.empty((batch, rows), dtype=torch.float16, device=device) for _ in pms]

    def run():
        for pm, y in zip(pms, ys):
            pm.gemv(x, y=y, y_fp16=True)

    return Workload(name or f"shape_{'v2a' if mode else 'v2'}_{rows}x{cols}_n{bits}_b{batch}",
                    {"workload": f"{rows}x{cols} {'V2a' if mode else 'V2'} N={bits}", "rows": rows, "cols": cols,
                     "mode": "V2a" if mode else "V2", "bits": bits, "outlier_rate": rate, "placement": placement,
                     "batch": batch, "copies": copies},
                    run, nb * copies, copies, copies, keep=[pms, x, ys],
                    sample=[(synth.to_host(q), synth.activations(batch, cols, 3))] if rows * cols <= (1 << 24) else [])


def gemm(mode: int, rows: int, cols: int, bits: int, rate: float, m: int, device="cuda", copies: Optional[int] = None) -> Workload:
    """The prefill form (xfp_gemm, tcgen05) with m rows of x on one matrix, cycled over distinct packed copies."""
    q = synth.random_quantized_torch(mode, rows, cols, bits, rate, seed=1, device=device)
    first = _pack(q, device)
    nb = _bytes_of(first, 0) + m * (cols * 2 + rows * 2)
    if copies is None:
        copies = max(2, int(2 * L2_BYTES // nb) + 1)
    blobs = [first.packed] + [first.packed.clone() for _ in range(copies - 1)]
    x = _x(m, cols, 3, device)
    ys = [torch.empty((m, rows), dtype=torch.float16, device=device) for _ in blobs]
    wss = [torch.zeros(xb.xfp_gemm_workspace_size(first.desc, m), dtype=torch.uint8, device=device) for _ in blobs]

    def run():
        for blob, y, ws in zip(blobs, ys, wss):
            xb.xfp_gemm(first.desc, blob, x, y, ws)

    return Workload(f"gemm_{'v2a' if mode else 'v2'}_{rows}x{cols}_n{bits}_m{m}",
                    {"workload": f"prefill form, {rows}x{cols} {'V2a' if mode else 'V2'} N={bits}, {m} rows of x",
                     "rows": rows, "cols": cols, "bits": bits, "outlier_rate": rate, "m": m, "copies": copies,
                     "flops_per_call": 2.0 * m * rows * cols},
                    run, nb * copies, copies, copies, keep=[blobs, x, ys, wss, first])


def pack_dequant(mode: int, rows: int, cols: int, bits: int, rate: float, device="cuda") -> Workload:
    """xfp_pack (unpacked tensors -> blob) followed by xfp_dequant (blob -> fp16 matrix) on one matrix; bytes: byte
    indices in and bit stream out for pack, blob in and fp16 matrix out for dequant, metadata both ways."""
    q = synth.random_quantized_torch(mode, rows, cols, bits, rate, seed=1, device=device)
    pm = _pack(q, device)
    d = pm.desc
    W = torch.empty((rows, cols), dtype=torch.float16, device=device)
    ocol = q.ocol.to(torch.int16) if q.ocol.numel() else torch.zeros(16, dtype=torch.int16, device=device)
    oval = q.oval if q.oval.numel() else torch.zeros(16, dtype=torch.int16, device=device)

    def run():
        xb.xfp_pack(d, q.idx, q.codebook, q.gid, q.gscale, q.gmid, q.rowptr, ocol, oval, pm.packed, pm.err_word)
        xb.xfp_dequant(d, pm.packed, W)

    meta = _bytes_of(pm, 0) - rows * cols * bits // 8
    nbytes = (rows * cols + rows * cols * bits // 8 + 2 * meta) + (rows * cols * bits // 8 + meta + rows * cols * 2)
    return Workload(f"pack_dequant_{rows}x{cols}_n{bits}", {"workload": f"xfp_pack + xfp_dequant, {rows}x{cols} N={bits}",
                                                            "rows": rows, "cols": cols, "bits": bits, "outlier_rate": rate},
                    run, nbytes, 2, 9, keep=[q, pm, W, ocol, oval])


def single(device="cuda") -> Workload:
    w = shape(0, 4096, 4096, 4, 0.003, device=device, name="single")
    w.config["workload"] = "single linear 4096x4096, V2 N=4, 0.3 % outliers (configuration 1)"
    return w


def moe(experts: int = 128, tokens: int = 64, bits: int = 3, device="cuda", distinct: int = 8) -> Workload:
    """Routed-MoE decode: every token-layer is two grouped launches over the token's 8 experts, the first storing
    SiLU(gate) * up, the second the routing-weighted sum ("MoE-native" dispatch)."""
    shapes = {"gate_up": (3072, 4096), "down": (4096, 1536)}
    packed, descs, nbytes = {}, {}, {}
    for name, (rows, cols) in shapes.items():
        base, lib = [], None
        for j in range(distinct):
            q = synth.random_quantized_torch(1, rows, cols, bits, 0.001, seed=100 + j, device=device, library=lib)
            lib = q.codebook                      # one library per projection, shared by the layer's experts
            base.append(_pack(q, device))
        pms = []
        for e in range(experts):
            b = base[e % distinct]
            pms.append(b if e < distinct else xb.PackedMatrix(b.desc, b.packed.clone(), b.workspace, b.err_word))
        packed[name] = pms
        d0 = pms[0].desc
        descs[name] = xb.XfpDesc(d0.mode, d0.rows, d0.cols, d0.bits, d0.group_size, d0.lib_size, d0.col_bits,
                                 max(p.desc.nnz for p in pms))
        nbytes[name] = _bytes_of(base[0])
    route = synth.moe_routing(tokens, experts, 8, seed=7)
    x_up = [_x(1, 4096, 40 + t, device) for t in range(tokens)]
    h = [torch.zeros((8, 1536), dtype=torch.float16, device=device) for _ in range(tokens)]
    y_out = [torch.empty((8, 4096), dtype=torch.float16, device=device) for _ in range(tokens)]
    ptrs = lambda ts: torch.tensor([t.data_ptr() for t in ts], dtype=torch.int64, device=device)
    gate_w = torch.full((8,), 0.125, dtype=torch.float32, device=device)
    args = []
    for t in range(tokens):
        ex = route[t]
        args.append((ptrs([packed["gate_up"][e].packed for e in ex]), ptrs([x_up[t]] * 8), ptrs([h[t][j] for j in range(8)]),
                     ptrs([packed["down"][e].packed for e in ex]), ptrs([y_out[t][j] for j in range(8)])))
    ws = {n: torch.zeros(8 * xb.xfp_packed_size(descs[n])[1], dtype=torch.uint8, device=device) for n in shapes}

    def run():
        for a in args:
            xb.xfp_gemv_grouped_epilogue(descs["gate_up"], 8, a[0], a[1], a[2], True, xb.XFP_EPI_SWIGLU, None, ws["gate_up"])
            xb.xfp_gemv_grouped_epilogue(descs["down"], 8, a[3], a[2], a[4], True, xb.XFP_EPI_COMBINE, gate_w, ws["down"])

    per_layer = 8 * (nbytes["gate_up"] + nbytes["down"])
    return Workload("moe", {"workload": "routed-MoE token-layer (configuration 3)", "mode": "V2a", "bits": bits,
                            "experts": experts, "top_k": 8, "tokens_per_step": tokens, "outlier_rate": 0.001,
                            "gate_up": "3072x4096", "down": "4096x1536", "lib_size": 32,
                            "launches": "two grouped launches per token-layer with fused SiLU*up and weighted-sum stores"},
                    run, per_layer * tokens, 16 * tokens, 2 * tokens, keep=[packed, x_up, h, y_out, args, ws, gate_w])


# ------------------------------------------------------------------------------------------------ timing

class GraphRunner:
    """One step of a workload captured as a CUDA graph on a stream of its own."""

    def __init__(self, w: Workload, device):
        self.w = w
        self.stream = torch.cuda.Stream(device=device)
        with torch.cuda.stream(self.stream):
            w.run()                              # first call of every kernel variant outside the capture
            self.stream.synchronize()
            self.graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.graph, stream=self.stream):
                w.run()
        self.stream.synchronize()

    def replay(self, n: int = 1):
        with torch.cuda.stream(self.stream):
            for _ in range(n):
                self.graph.replay()

    def ramp(self, seconds: float) -> float:
        """Replay for a fixed wall time so that the SM clock has left its idle state; returns milliseconds spent."""
        import time
        t0 = time.perf_counter()
        while time.perf_counter() - t0 < seconds:
            self.replay(4)
            self.stream.synchronize()
        return (time.perf_counter() - t0) * 1e3

    def time(self, steps: int, warmup: int, min_region_s: float = 0.25, barrier: Optional[Callable] = None):
        """(ms per step, replays per step R, region ms): `warmup` steps, then steps * R replays between two events on
        the launching stream, R chosen so that the region lasts at least min_region_s."""
        self.replay(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(self.stream):
            e0.record(self.stream)
            self.graph.replay()
            e1.record(self.stream)
        self.stream.synchronize()
        est = max(e0.elapsed_time(e1), 1e-3) * 1e-3
        R = max(1, int(math.ceil(min_region_s / (steps * est))))
        self.replay(warmup)
        self.stream.synchronize()
        if barrier:
            barrier()
        with torch.cuda.stream(self.stream):
            e0.record(self.stream)
            for _ in range(steps * R):
                self.graph.replay()
            e1.record(self.stream)
        self.stream.synchronize()
        if barrier:
            barrier()
        region = e0.elapsed_time(e1)
        return region / (steps * R), R, region


def profile_launches(w: Workload, launches: int, device) -> None:
    """`launches` steps of the workload, each after a 512 MB fill that evicts the L2: the target of profiler captures."""
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=device)
    w.run()
    torch.cuda.synchronize(device)
    for _ in range(launches):
        flush.fill_(1)
        w.run()
    torch.cuda.synchronize(device)


def parse(spec: str, device="cuda", **kw) -> Workload:
    """Workload from a name: stack_v2 | stack_v2a | attention | single | moe |
    shape:MODE:ROWS:COLS:BITS:RATE[:BATCH[:PLACEMENT[:COPIES]]] | gemm:MODE:ROWS:COLS:BITS:RATE:M[:COPIES] |
    packdq:MODE:ROWS:COLS:BITS:RATE  (MODE 0 = V2, 1 = V2a)."""
    if spec in ("stack_v2", "stack_v2a"):
        return stack(1 if spec.endswith("a") else 0, device=device, **kw)
    if spec == "attention":
        return attention(device=device)
    if spec == "attention_grouped":
        return attention_grouped(device=device)
    if spec == "single":
        return single(device=device)
    if spec == "moe":
        return moe(device=device)
    if spec.startswith("shape:"):
        f = spec.split(":")[1:]
        mode, rows, cols, bits = (int(v) for v in f[:4])
        return shape(mode, rows, cols, bits, float(f[4]), int(f[5]) if len(f) > 5 else 1,
                     f[6] if len(f) > 6 else "uniform", device=device, copies=int(f[7]) if len(f) > 7 else None)
    if spec.startswith("gemm:"):      # gemm:MODE:ROWS:COLS:BITS:RATE:M[:COPIES]
        f = spec.split(":")[1:]
        return gemm(int(f[0]), int(f[1]), int(f[2]), int(f[3]), float(f[4]), int(f[5]), device=device,
                    copies=int(f[6]) if len(f) > 6 else None)
    if spec.startswith("packdq:"):    # packdq:MODE:ROWS:COLS:BITS:RATE
        f = spec.split(":")[1:]
        return pack_dequant(int(f[0]), int(f[1]), int(f[2]), int(f[3]), float(f[4]), device=device)
    raise ValueError(f"unknown workload {spec!r}")
