#!/usr/bin/env python
"""Benchmark of the fused XFP decode GEMV on B200.

Headline workload: the mixed-bit 48-layer decoder linear sweep at batch 1 in V2 storage -- per layer q/k/v/o
4096 x 4096 plus an MLP of 12288 x 4096 and 4096 x 12288, bit width per layer from {2..6}, outlier rate from
[0, 2 %] -- the largest single-GPU configuration: 288 fused GEMV calls and about 4.4 GB of packed weights per token,
far beyond the 126 MB L2, so every call streams its weights from HBM.  One step = one token through the stack,
replayed as one CUDA graph.

Prints ONE JSON line: effective GB/s over the algorithmic bytes (indices, codebooks, outlier values and columns, row
pointers, x, y), microseconds per call, the HBM roofline of the GEMV kernels, the same step measured end to end from
pinned host buffers through xfp_gemv_host, the clocks sampled during the timed regions, and -- at one GPU -- a
`configs` object with the other configurations (single 4096 x 4096 layer, dense attention blocks, routed-MoE
token-layer in V2a with fused stores, the same stack in V2a, 8192 x 8192 and 28672 x 8192 in V2 and V2a) and the CPU
oracle timed on a bounded sample.

    python bench.py [--gpus N] [--steps K] [--warmup W]
    python bench.py --impl reference ...          the CPU oracle alone on a bounded sample of the headline workload
    python bench.py --workload NAME               time one workload alone and print its entry (see workloads.parse)
    python bench.py --workload NAME --launches n  n cold launches of it and no timing: the target of profiler captures
    python bench.py --encoder                     Algorithm 1 on one attention projection on the GPU, oracle beside it
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
METRIC = "fused XFP GEMV effective GB/s at batch 1"
MIN_REGION_S = 0.25
# dram__bytes_read.sum + dram__bytes_write.sum per launch divided by the algorithmic bytes of that launch, from the
# ncu captures of the batch-1 V2 kernel summarised under profiles/ (gemv_lane_v2_4096x4096.md: 9.62 MB against 9.16 MB
# = 1.05; gemv_lane_v2_28672x8192.md: 125.8 MB against 121.4 MB = 1.04).  The stack's 288 launches are those kernels
# on 25-75 MB matrices; its traffic is scaled from them by bytes (traffic grows with the matrix, nothing is re-read).
NCU_TRAFFIC_RATIO = {"stack_v2": 1.045, "shape_v2_28672x8192_n4_b1": 1.036, "single": 1.05}


def block_spec(layer: int):
    """(name, bits, seed) of the four projections of one dense-attention block; bits seeded from {4, 5}."""
    rng = np.random.default_rng(1000 + layer)
    bits = rng.integers(4, 6, size=4)
    return [(n, int(b), 10 + 4 * layer + j) for j, (n, b) in enumerate(zip("qkvo", bits))]


def algorithmic_bytes(q) -> int:
    """Bytes one batch-1 call on the unpacked tensors `q` must move (fp16 y)."""
    from paper_2605_14844_b200.workloads import algorithmic_bytes as ab
    return ab(q.mode, q.rows, q.cols, q.bits, q.nnz, q.lib_size, q.group_size)


class ClockSampler:
    """nvidia-smi clocks and throttle reasons while the timed regions run."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None
        self.marks = []   # (first row, last row) of every timed region

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([f.strip() for f in line.split(",")])

    def region(self):
        """Context manager marking the samples that arrive while a timed region runs."""
        sampler = self

        class _R:
            def __enter__(self):
                self.a = len(sampler.rows)

            def __exit__(self, *exc):
                sampler.marks.append((self.a, len(sampler.rows)))
        return _R()

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        inside = [r for a, b in self.marks for r in self.rows[a:b]]
        sm, mx, reasons, power = [], [], set(), []
        for r in inside:
            try:
                sm.append(float(r[1])); mx.append(float(r[2])); power.append(float(r[3]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "samples_total": len(self.rows),
                "power_w_max": max(power) if power else None,
                "how": "nvidia-smi every 50 ms; only samples that arrived inside a timed region are counted"}


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


def time_oracle(sample, budget_s: float, what: str):
    """The oracle's fp64 GEMV over `sample` = [(QuantTensors on the host, x16)], repeated for about budget_s seconds."""
    from oracle import xfp_oracle as xo
    oms = [oracle_matrix(q) for q, _ in sample]
    xs = [x for _, x in sample]
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
    nbytes = reps * sum(algorithmic_bytes(q) for q, _ in sample)
    return {"value": nbytes / dt / 1e9, "unit": "GB/s", "cores": xo.threads(), "kind": "oracle",
            "us_per_call": dt / calls * 1e6, "sample": f"{calls} fp64 GEMV calls over {what} ({dt:.1f} s)"}


def reference_sample():
    """The first decoder layer of the headline stack on the host (its six linears), for the CPU oracle."""
    from paper_2605_14844_b200 import synth
    from paper_2605_14844_b200 import workloads as wl
    bits, rate = wl.stack_spec()[0]
    out = []
    for j, (rows, cols) in enumerate(wl.STACK_SHAPES):
        q = synth.to_host(synth.random_quantized_torch(0, rows, cols, bits, rate, seed=5000 + j, device="cpu"))
        out.append((q, synth.activations(1, cols, 900 + cols)))
    return out, bits, rate


def run_reference(args, rank: int):
    if rank != 0:
        return
    from oracle import xfp_oracle as xo
    sample, bits, rate = reference_sample()
    oms = [oracle_matrix(q) for q, _ in sample]
    step_bytes = sum(algorithmic_bytes(q) for q, _ in sample)
    for _ in range(args.warmup):
        for m, (_, x) in zip(oms, sample):
            xo.gemv(m, x)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        for m, (_, x) in zip(oms, sample):
            xo.gemv(m, x)
    dt = time.perf_counter() - t0
    val = args.steps * step_bytes / dt / 1e9
    what = (f"layer 0 of the 48-layer stack (its six linears, N={bits}, {rate * 100:.1f} % outliers) per step, "
            "fp64 CPU oracle")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "us_per_call": dt / (args.steps * len(oms)) * 1e6,
        "config": {"workload": "48-layer mixed-bit decoder linear sweep (configuration 4)", "mode": "V2", "batch": 1,
                   "sample": what},
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": xo.threads(), "kind": "oracle", "sample": what},
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


def entry_of(w, ms_per_step: float, R: int, region_ms: float, peak: float) -> dict:
    """The per-configuration record: microseconds per call, effective GB/s, fraction of the HBM roofline."""
    gbs = w.bytes_per_step / (ms_per_step * 1e-3) / 1e9
    return {"config": w.config, "us_per_call": ms_per_step * 1e3 / w.calls_per_step,
            "us_per_launch": ms_per_step * 1e3 / w.launches_per_step, "ms_per_step": ms_per_step,
            "calls_per_step": w.calls_per_step, "launches_per_step": w.launches_per_step,
            "bytes_per_step": w.bytes_per_step, "GBs": gbs, "frac": gbs / peak, "frac_of_nominal_8000": gbs / NOMINAL_HBM_GBS,
            "replays_per_step": R, "region_ms": region_ms}


EXTRA_CONFIGS = (
    ("config1_single_4096x4096_v2_n4", "single"),
    ("config2_attention_blocks_v2", "attention"),
    ("config2_attention_blocks_v2_grouped_qkv", "attention_grouped"),
    ("config3_moe_token_layer_v2a_n3", "moe"),
    ("config4_stack_v2a", "stack_v2a"),
    ("config5_8192x8192_v2_n4", "shape:0:8192:8192:4:0.003"),
    ("config5_8192x8192_v2a_n4", "shape:1:8192:8192:4:0.003"),
    ("config5_28672x8192_v2_n4", "shape:0:28672:8192:4:0.003"),
    ("config5_28672x8192_v2a_n4", "shape:1:28672:8192:4:0.003"),
    # the batch axis of configuration 5: 8 rows of x (the other batch sizes: `--workload shape:...:BATCH`)
    ("config5_8192x8192_v2_n4_batch8", "shape:0:8192:8192:4:0.003:8"),
    ("config5_28672x8192_v2_n4_batch8", "shape:0:28672:8192:4:0.003:8"),
    ("config5_28672x8192_v2a_n4_batch8", "shape:1:28672:8192:4:0.003:8"),
)


def run_xfp(args, rank: int, world: int):
    import torch
    import paper_2605_14844_b200 as xfp  # noqa: F401  (fails loudly when libxfp.so is missing)
    from paper_2605_14844_b200 import workloads as wl

    xfp.load_library()
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    peak, peak_kind = measured_peak()
    # ---- the headline workload (same seeds on every rank: replicas, no data-path collective)
    t_build = time.perf_counter()
    w = wl.parse(args.workload or "stack_v2", device=dev, **({"with_host": True, "n_sample": 6}
                                                             if (args.workload or "stack_v2").startswith("stack") else {}))
    if args.launches:
        wl.profile_launches(w, args.launches, dev)
        print(json.dumps({"workload": w.name, "launches": args.launches * w.launches_per_step, "mode": "cold launches for a profiler"}))
        return
    runner = wl.GraphRunner(w, dev)
    build_s = time.perf_counter() - t_build
    sampler = ClockSampler(local)
    sampler.start()
    ramp_ms = runner.ramp(0.6)                     # clock ramp, reported apart from the warm-up steps
    with sampler.region():
        ms_per_step, R, region_ms = runner.time(args.steps, max(args.warmup, 3), MIN_REGION_S, barrier)

    # ---- end to end through the C ABI with host buffers (pinned x in, y out, every call), one graph per step
    e2e_ms = None
    if w.host_step is not None:
        s = runner.stream
        with torch.cuda.stream(s):
            w.host_step(s)
            s.synchronize()
            graph_host = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph_host, stream=s):
                w.host_step(s)
            for _ in range(max(args.warmup, 3)):
                graph_host.replay()
            s.synchronize()
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n_e2e = args.steps * R
            with sampler.region():
                e0.record(s)
                for _ in range(n_e2e):
                    graph_host.replay()
                e1.record(s)
                s.synchronize()
            barrier()
            e2e_ms = e0.elapsed_time(e1) / n_e2e
        del graph_host

    ms_per_step, e2e_max = max_over_ranks([ms_per_step, e2e_ms or 0.0], dist, dev)
    head = entry_of(w, ms_per_step, R, region_ms, peak)
    sample_head = w.sample

    class Meta:   # what the line needs of the headline workload once its device tensors are released
        name, config, bytes_per_step, calls_per_step = w.name, w.config, w.bytes_per_step, w.calls_per_step
        launches_per_step, h2d_bytes, d2h_bytes = w.launches_per_step, w.h2d_bytes, w.d2h_bytes
    w = runner = None

    # ---- the other configurations (one GPU only: they are records, not the scaling curve)
    configs = {}
    if world == 1 and not args.workload and not args.no_configs:
        torch.cuda.empty_cache()
        for key, spec in EXTRA_CONFIGS:
            try:
                wc = wl.parse(spec, device=dev)
                rc = wl.GraphRunner(wc, dev)
                rc.ramp(0.1)
                with sampler.region():
                    ms, Rc, reg = rc.time(max(3, args.steps // 4), 3, MIN_REGION_S)
                configs[key] = entry_of(wc, ms, Rc, reg, peak)
            except Exception as e:  # a configuration that fails is reported, not hidden
                configs[key] = {"error": f"{type(e).__name__}: {e}"}
            wc = rc = None
            torch.cuda.empty_cache()
    clocks = sampler.stop()
    clocks["ramp_ms"] = ramp_ms

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    w = Meta
    value = aggregate_value(w.bytes_per_step, world, ms_per_step)
    ratio = NCU_TRAFFIC_RATIO.get(w.name)
    out = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "us_per_call": head["us_per_call"],
        "config": dict(w.config, calls_per_step=w.calls_per_step, bytes_per_step=w.bytes_per_step,
                       replays_per_step=R, region_ms=region_ms, build_s=build_s,
                       l2="the weights of a step (%.2f GB) exceed the 126 MB L2 many times over" % (w.bytes_per_step / 1e9)
                       if w.bytes_per_step > 4 * wl.L2_BYTES else "distinct packed copies, more than twice the L2, are cycled",
                       launch="one CUDA graph per step; a timed step is %d replays" % R),
        "roofline": {"bound": "hbm", "achieved": head["GBs"], "peak": peak, "unit": "GB/s", "frac": head["frac"],
                     "peak_kind": peak_kind, "frac_of_nominal_8000": head["frac_of_nominal_8000"],
                     "traffic": None if ratio is None else ratio * w.bytes_per_step / w.launches_per_step,
                     "bytes_per_launch": w.bytes_per_step / w.launches_per_step,
                     "kernel": "the fused GEMV kernels of a step (average over its launches)"},
        "gpu_launches": (args.steps * R + max(args.warmup, 3)) * w.launches_per_step,
        "clocks": clocks,
    }
    if e2e_ms is not None:
        out["e2e"] = {"value": aggregate_value(w.bytes_per_step, world, e2e_max), "unit": "GB/s",
                      "h2d_bytes_per_step": w.h2d_bytes, "d2h_bytes_per_step": w.d2h_bytes,
                      "us_per_call": e2e_max * 1e3 / w.calls_per_step,
                      "how": "xfp_gemv_host per call (pinned x in, fused GEMV, pinned y out), the step captured once as a "
                             "CUDA graph and replayed"}
    if configs:
        out["configs"] = configs
    if world == 1 and not args.no_cpu_baseline and sample_head:
        out["cpu_baseline"] = time_oracle(sample_head, args.cpu_seconds, "the six linears of layer 0 of the stack")
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


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
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="xfp", choices=["xfp", "reference"])
    ap.add_argument("--workload", default=None, help="time this workload instead of the headline (workloads.parse)")
    ap.add_argument("--launches", type=int, default=0, help="with --workload: cold launches for a profiler, no timing")
    ap.add_argument("--no-configs", action="store_true", help="headline only")
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
