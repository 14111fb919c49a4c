#!/usr/bin/env python
"""Benchmark of the fused XFP decode GEMV on B200.

Workload (the dense-attention configuration): a stack of `--layers` attention blocks, each with
four 4096 x 4096 V2 projections (q, k, v, o) whose bit width is drawn from {4, 5} and whose
~0.9 % fp16 outliers sit in heavy outlier columns; batch 1, fp16 activations, fp16 outputs.
One step = one token through every block = 4 * layers fused GEMV calls, replayed as one CUDA
graph.  The stack (~40 MB per block) is larger than the 126 MB L2, so every call streams its
weights from HBM.

Prints one JSON line: effective GB/s over the algorithmic bytes (indices, codebooks, outlier
values and columns, row pointers, x, y), microseconds per call, the HBM roofline of the GEMV
kernel, the same measured end to end from host buffers, and the CPU oracle timed beside it.

`--impl reference` times the CPU oracle alone on the same workload (bounded sample per step).

`--encoder` is a separate, optional measurement (not the headline line): Algorithm 1 on one 4096 x 4096
attention projection (float weights with heavy outlier columns -> extraction, per-channel Lloyd over the
candidates {4, 5}, residual, cosine gate) through xfp_quantize on the GPU, with the oracle's encoder timed
beside it on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

ROWS = COLS = 4096
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the two GEMV kernels of this workload, from
# the ncu captures summarised in profiles/gemv_pair_attention_4096x4096.md (bits -> bytes)
NCU_TRAFFIC_BYTES_PER_LAUNCH = {4: 9623296, 5: 11855616}


def block_spec(layer: int):
    """(name, bits, seed) of the four projections of one block; bits seeded from {4, 5}."""
    rng = np.random.default_rng(1000 + layer)
    bits = rng.integers(4, 6, size=4)
    return [(n, int(b), 10 + 4 * layer + j) for j, (n, b) in enumerate(zip("qkvo", bits))]


def make_matrix(bits: int, seed: int):
    from paper_2605_14844_b200 import synth
    return synth.random_quantized(0, ROWS, COLS, bits, 0.009, seed, placement="clustered")


def algorithmic_bytes(q) -> int:
    E = 1 << q.bits
    b = q.rows * q.cols * q.bits // 8                    # packed indices
    b += (q.rows if q.mode == 0 else q.lib_size) * E * 2  # codebooks / library
    if q.mode == 1:
        b += q.rows * (q.cols // q.group_size) * 5        # id u8 + scale fp16 + mid fp16 per group
    b += q.nnz * 4 + (q.rows + 1) * 4                     # outlier value + u16 column, row pointers
    b += q.cols * 2 + q.rows * 2                          # x fp16, y fp16
    return b


class ClockSampler:
    """nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([f.strip() for f in line.split(",")])

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except (OSError, KeyError, ValueError):
        return FALLBACK_HBM_GBS, "fallback"


def oracle_matrix(q):
    from oracle import xfp_oracle as xo
    return xo.QuantizedMatrix(q.mode, q.rows, q.cols, q.bits, q.idx, q.codebook, q.rowptr, q.ocol, q.oval,
                              group_size=q.group_size, lib_size=q.lib_size, gid=q.gid, gscale=q.gscale, gmid=q.gmid)


def time_oracle(mats, xs, budget_s: float):
    """Repeat the oracle's fp64 GEMV over `mats` until about budget_s seconds are spent."""
    from oracle import xfp_oracle as xo
    oms = [oracle_matrix(q) for q in mats]
    t0 = time.perf_counter()
    xo.gemv(oms[0], xs[0])
    t1 = time.perf_counter() - t0
    reps = max(1, min(200, int(budget_s / max(t1 * len(oms), 1e-6))))
    t0 = time.perf_counter()
    for _ in range(reps):
        for m, x in zip(oms, xs):
            xo.gemv(m, x)
    dt = time.perf_counter() - t0
    calls = reps * len(oms)
    nbytes = reps * sum(algorithmic_bytes(q) for q in mats)
    return {"value": nbytes / dt / 1e9, "unit": "GB/s", "cores": xo.threads(), "kind": "oracle",
            "us_per_call": dt / calls * 1e6,
            "sample": f"{calls} fp64 GEMV calls over the q/k/v/o projections of block 0 ({dt:.1f} s)"}


def run_reference(args, rank: int):
    if rank != 0:
        return
    from paper_2605_14844_b200 import synth
    spec = block_spec(0)
    mats = [make_matrix(b, s) for _, b, s in spec]
    xs = [synth.activations(1, COLS, seed=900 + j) for j in range(4)]
    from oracle import xfp_oracle as xo
    oms = [oracle_matrix(q) for q in mats]
    step_bytes = sum(algorithmic_bytes(q) for q in mats)
    for _ in range(args.warmup):
        for m, x in zip(oms, xs):
            xo.gemv(m, x)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        for m, x in zip(oms, xs):
            xo.gemv(m, x)
    dt = time.perf_counter() - t0
    val = args.steps * step_bytes / dt / 1e9
    sample = "one attention block (4 projections) per step, fp64 CPU oracle"
    print(json.dumps({
        "impl": "reference", "metric": "fused XFP GEMV effective GB/s at batch 1", "value": val, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "us_per_call": dt / (args.steps * 4) * 1e6,
        "config": {"workload": "attention_block_v2", "rows": ROWS, "cols": COLS, "bits": [b for _, b, _ in spec],
                   "batch": 1, "sample": sample},
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": xo.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (the timed region of a multi-GPU run is
    as long as its slowest rank); identity when torch.distributed is not initialised."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_value(step_bytes: int, world: int, ms_per_step: float) -> float:
    """Whole-job GB/s of `world` replicas that each move step_bytes per step (weak scaling)."""
    return world * step_bytes / (ms_per_step * 1e-3) / 1e9


def run_xfp(args, rank: int, world: int):
    import torch
    import paper_2605_14844_b200 as xfp
    from paper_2605_14844_b200 import synth

    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    # ---- build the stack (same seeds on every rank: replicas, no data-path collective)
    mats, pms, names = [], [], []
    for layer in range(args.layers):
        for name, bits, seed in block_spec(layer):
            q = make_matrix(bits, seed)
            pm = xfp.pack_tensors(q, device=dev, col_bits=16)
            if layer == 0:
                mats.append(q)
            else:
                q.idx = None  # keep host memory small; sizes are kept below
            pms.append(pm); names.append((layer, name, bits, algorithmic_bytes_from(pm, q)))
    torch.cuda.synchronize()
    assert all(int(p.err_word.item()) == 0 for p in pms)
    n_calls = len(pms)
    step_bytes = sum(n[3] for n in names)

    x16 = [synth.activations(1, COLS, seed=900 + j) for j in range(n_calls)]
    xd = [torch.from_numpy(x.view(np.int16)).to(dev).view(torch.float16) for x in x16]
    yd = [torch.empty((1, ROWS), dtype=torch.float16, device=dev) for _ in range(n_calls)]

    def step():
        for pm, x, y in zip(pms, xd, yd):
            pm.gemv(x, y=y, y_fp16=True)

    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        step()                      # first call sets kernel attributes; keep it out of the capture
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            step()
        def barrier():
            if dist is not None:
                dist.barrier()
            torch.cuda.synchronize()

        # the clock sampler needs a moment to come up: warm up until it has delivered a sample (at
        # least the requested warm-up steps, at most ~2 s), so that the timed region is covered
        sampler = ClockSampler(local)
        sampler.start()
        t_w = time.perf_counter()
        n_warm = 0
        while n_warm < max(args.warmup, 3) or (len(sampler.rows) < 2 and time.perf_counter() - t_w < 2.0):
            graph.replay()
            n_warm += 1
            if n_warm % 64 == 0:
                stream.synchronize()
        stream.synchronize()
        n_before = len(sampler.rows)
        barrier()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        ev[0].record(stream)
        for i in range(args.steps):
            graph.replay()
            ev[i + 1].record(stream)
        barrier()
        time.sleep(0.12)   # one more sampling period, so a short timed region still sees a sample taken under load
        clocks = sampler.stop()
        clocks["samples_before_timed_region"] = n_before
        clocks["warmup_steps_run"] = n_warm
        total_ms = ev[0].elapsed_time(ev[-1])
        per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]

        # ---- end to end through the C ABI with host buffers (pinned x in, y out, every call)
        xh = [torch.from_numpy(x.view(np.int16)).pin_memory() for x in x16]
        yh = [torch.empty((1, ROWS), dtype=torch.float16).pin_memory() for _ in range(n_calls)]

        def step_host():
            for pm, a, b, c, d in zip(pms, xh, xd, yh, yd):
                xfp.xfp_gemv_host(pm.desc, pm.packed, a, b, 1, c, d, True, pm.workspace, stream)

        for _ in range(3):
            step_host()
        stream.synchronize()
        # the step's host copies and launches are captured once and replayed: every replay copies the 32
        # x vectors from pinned host memory, runs the 32 fused GEMVs and copies the 32 results back
        graph_host = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph_host, stream=stream):
            step_host()
        for _ in range(3):
            graph_host.replay()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            graph_host.replay()
        e1.record(stream)
        barrier()
        e2e_ms = e0.elapsed_time(e1)

    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], dist, dev)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    ms_per_step = total_ms / args.steps
    value = aggregate_value(step_bytes, world, ms_per_step)
    e2e_val = aggregate_value(step_bytes, world, e2e_ms / args.steps)
    peak, peak_kind = measured_peak()
    per_gpu = step_bytes / (ms_per_step * 1e-3) / 1e9
    out = {
        "metric": "fused XFP GEMV effective GB/s at batch 1", "value": value, "unit": "GB/s", "n_gpus": world,
        "steps": args.steps, "warmup": n_warm, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "us_per_call": ms_per_step * 1e3 / n_calls,
        "ms_per_step_median": statistics.median(per_step),
        "config": {"workload": "attention_block_v2", "layers": args.layers, "calls_per_step": n_calls, "rows": ROWS,
                   "cols": COLS, "bits": [n[2] for n in names[:4]], "mode": "V2", "batch": 1, "outlier_rate": 0.009,
                   "bytes_per_step": step_bytes, "l2": "weights of a step (%.0f MB) exceed L2; none re-read before "
                   "126 MB of other weights passed" % (step_bytes / 1e6), "launch": "one CUDA graph per step"},
        "roofline": {"bound": "hbm", "achieved": per_gpu, "peak": peak, "unit": "GB/s", "frac": per_gpu / peak,
                     "peak_kind": peak_kind, "frac_of_nominal_8000": per_gpu / NOMINAL_HBM_GBS,
                     "traffic": sum(NCU_TRAFFIC_BYTES_PER_LAUNCH[n[2]] for n in names) / n_calls, "bytes_per_launch": step_bytes / n_calls,
                     "kernel": "gemv (all calls of a step)"},
        "e2e": {"value": e2e_val, "unit": "GB/s", "h2d_bytes_per_step": n_calls * COLS * 2,
                "d2h_bytes_per_step": n_calls * ROWS * 2, "us_per_call": e2e_ms / args.steps * 1e3 / n_calls,
                "how": "xfp_gemv_host per projection (pinned x in, fused GEMV, pinned y out), the step captured once "
                       "as a CUDA graph and replayed"},
        "gpu_launches": args.steps * n_calls,
        "clocks": clocks,
    }
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = time_oracle(mats, x16[:4], args.cpu_seconds)
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def algorithmic_bytes_from(pm, q) -> int:
    d = pm.desc
    E = 1 << d.bits
    return (d.rows * d.cols * d.bits // 8 + d.rows * E * 2 + d.nnz * 4 + (d.rows + 1) * 4 + d.cols * 2 + d.rows * 2)


def run_encoder(args):
    """One JSON line: the GPU encoder on a dense-attention projection, the oracle's encoder beside it."""
    import torch
    from paper_2605_14844_b200 import quant_binding as qb
    from paper_2605_14844_b200 import synth
    W = synth.attention_weights(10, ROWS, COLS)
    Wd = torch.from_numpy(W).cuda()
    cands, tau = (4, 5), 0.96
    buf = qb.QuantBuffers(ROWS, COLS, 0, max(cands), 0, int(0.02 * W.size))
    params = qb.XfpQuantParams(0, 0, 4.0, 0.02, 0.0, 20, 0)
    walls = []
    for it in range(args.warmup + 5):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        res = qb.xfp_quantize(0, Wd, params, cands, tau, buf)
        torch.cuda.synchronize()
        if it >= args.warmup:
            walls.append(time.perf_counter() - t0)
    gpu_s = statistics.median(walls)
    line = {"metric": "XFP encoder (Algorithm 1, V2) weights per second", "value": W.size / gpu_s / 1e6,
            "unit": "Mweights/s", "ms_per_matrix": gpu_s * 1e3, "n_gpus": 1, "higher_is_better": True,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": "one 4096x4096 attention projection, heavy outlier columns, candidates {4,5}, "
                                   "tau 0.96, 20 Lloyd rounds", "bits_chosen": int(res.bits), "nnz": int(res.nnz),
                       "median_cos": res.median_cos}}
    if not args.no_cpu_baseline:
        from oracle import xfp_oracle as xo
        t0 = time.perf_counter()
        ref = xo.auto_select(W, "attention", cands, tau_strict=tau, iters=20)
        cpu_s = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": W.size / cpu_s / 1e6, "unit": "Mweights/s", "cores": xo.threads(),
                                "kind": "oracle", "sample": "the same matrix, whole", "seconds": cpu_s,
                                "same_bits": int(ref.bits) == int(res.bits), "same_nnz": ref.nnz == int(res.nnz)}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="xfp", choices=["xfp", "reference"])
    ap.add_argument("--layers", type=int, default=8)
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--encoder", action="store_true", help="time the GPU encoder instead of the decode path")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.encoder:
        if rank == 0:
            run_encoder(args)
    elif args.impl == "reference":
        run_reference(args, rank)
    else:
        run_xfp(args, rank, world)


if __name__ == "__main__":
    main()
