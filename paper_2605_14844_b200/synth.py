"""Seeded synthetic inputs for the XFP decode path.

This module only draws numbers: weight matrices shaped like the paper's layers, activation
vectors, MoE routing, and ready-made quantised tensors (indices, codebooks, group metadata,
CSR outliers) with the sizes and sparsity structure of the paper's workloads.  It holds none
of the method's arithmetic (no Lloyd, no dequantisation, no packing), so both the CPU oracle's
tests and the CUDA path may use it.

All draws use numpy's PCG64 through ``default_rng(seed)``; the weight, outlier-position,
activation and routing seeds are kept distinct by the callers.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np

SIGMA0 = 0.02  # bulk standard deviation of the synthetic weights


# ---------------------------------------------------------------- dense fp32 weights

def gaussian_weights(rows: int, cols: int, seed: int, sigma: float = SIGMA0) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((rows, cols), dtype=np.float32) * np.float32(sigma))


def plant_uniform_outliers(W: np.ndarray, rate: float, seed: int, lo: float = 10.0, hi: float = 49.0,
                           sigma: float = SIGMA0) -> np.ndarray:
    """Overwrite a `rate` fraction of positions (uniform, without replacement) with +-U(lo,hi)*sigma."""
    rng = np.random.default_rng(seed)
    n = W.size
    m = int(round(rate * n))
    if m == 0:
        return W
    pos = rng.choice(n, size=m, replace=False)
    mag = rng.uniform(lo, hi, size=m) * sigma
    sgn = rng.integers(0, 2, size=m) * 2 - 1
    W.reshape(-1)[pos] = (mag * sgn).astype(np.float32)
    return W


def plant_column_outliers(W: np.ndarray, rate: float, seed: int, fill: float = 0.5, lo: float = 10.0,
                          hi: float = 49.0, sigma: float = SIGMA0) -> np.ndarray:
    """Heavy outlier columns: about `rate` of all weights, concentrated in rate/fill of the input
    columns, each hot column hit with probability `fill` per row."""
    rng = np.random.default_rng(seed)
    rows, cols = W.shape
    n_hot = max(1, int(round(rate * cols / fill))) if rate > 0 else 0
    if n_hot == 0:
        return W
    hot = np.sort(rng.choice(cols, size=n_hot, replace=False))
    hit = rng.random((rows, n_hot)) < fill
    mag = rng.uniform(lo, hi, size=(rows, n_hot)) * sigma
    sgn = rng.integers(0, 2, size=(rows, n_hot)) * 2 - 1
    sub = W[:, hot]
    sub[hit] = (mag * sgn).astype(np.float32)[hit]
    W[:, hot] = sub
    return W


def config1_weights(seed: int = 1, rows: int = 4096, cols: int = 4096) -> np.ndarray:
    """Single linear layer: N(0, 0.02^2) bulk with 0.3 % of entries at 10-49 sigma."""
    W = gaussian_weights(rows, cols, seed)
    return plant_uniform_outliers(W, 0.003, seed + 1000)


def attention_weights(seed: int, rows: int = 4096, cols: int = 4096, rate: float = 0.01) -> np.ndarray:
    """Dense-attention projection: Gaussian bulk with heavy outlier columns (1 % of weights)."""
    W = gaussian_weights(rows, cols, seed)
    return plant_column_outliers(W, rate, seed + 1000)


def activations(batch: int, cols: int, seed: int) -> np.ndarray:
    """x ~ N(0,1) rounded to fp16; returned as fp16 bit patterns [batch, cols] (uint16)."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((batch, cols), dtype=np.float32).astype(np.float16)
    return x.view(np.uint16)


def moe_routing(tokens: int, experts: int = 128, top_k: int = 8, seed: int = 7) -> np.ndarray:
    """Per token the top_k experts by seeded Gaussian logits; int32 [tokens, top_k], ascending ids."""
    rng = np.random.default_rng(seed)
    logits = rng.standard_normal((tokens, experts))
    top = np.argsort(-logits, axis=1, kind="stable")[:, :top_k]
    return np.sort(top, axis=1).astype(np.int32)


# ---------------------------------------------------------------- ready-made quantised tensors

@dataclass
class QuantTensors:
    """Unpacked XFP tensors (host numpy), the input of xfp_pack."""
    mode: int                      # 0 = V2, 1 = V2a
    rows: int
    cols: int
    bits: int
    idx: np.ndarray                # uint8 [rows, cols]
    codebook: np.ndarray           # uint16 fp16 bits: V2 [rows, 2^N]; V2a [L, 2^N]
    rowptr: np.ndarray             # int32 [rows+1]
    ocol: np.ndarray               # int32 [nnz]
    oval: np.ndarray               # uint16 [nnz]
    group_size: int = 128
    lib_size: int = 0
    gid: Optional[np.ndarray] = None
    gscale: Optional[np.ndarray] = None
    gmid: Optional[np.ndarray] = None

    @property
    def nnz(self) -> int:
        return int(self.rowptr[-1])


def _f16bits(a: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(a.astype(np.float16)).view(np.uint16)


def random_csr(rows: int, cols: int, rate: float, seed: int, placement: str = "uniform", fill: float = 0.5,
               lo: float = 10.0, hi: float = 49.0, sigma: float = SIGMA0):
    """Outlier CSR with about `rate` of all positions: 'uniform' scatters them, 'clustered' puts
    them in rate/fill hot columns, 'one_row' gives every outlier to a single row."""
    rng = np.random.default_rng(seed)
    if rate <= 0:
        return np.zeros(rows + 1, np.int32), np.zeros(0, np.int32), np.zeros(0, np.uint16)
    if placement == "uniform":
        counts = rng.binomial(cols, rate, size=rows)
        colsel = [np.sort(rng.choice(cols, size=c, replace=False)) for c in counts]
    elif placement == "clustered":
        n_hot = max(1, int(round(rate * cols / fill)))
        hot = np.sort(rng.choice(cols, size=n_hot, replace=False))
        hit = rng.random((rows, n_hot)) < fill
        colsel = [hot[hit[i]] for i in range(rows)]
    elif placement == "one_row":
        n = min(cols, max(1, int(round(rate * rows * cols))))
        r = int(rng.integers(0, rows))
        colsel = [np.zeros(0, np.int64)] * rows
        colsel[r] = np.sort(rng.choice(cols, size=n, replace=False))
    else:
        raise ValueError(placement)
    rowptr = np.zeros(rows + 1, np.int32)
    rowptr[1:] = np.cumsum([len(c) for c in colsel])
    ocol = np.concatenate(colsel).astype(np.int32) if rowptr[-1] else np.zeros(0, np.int32)
    nnz = int(rowptr[-1])
    mag = rng.uniform(lo, hi, size=nnz) * sigma
    sgn = rng.integers(0, 2, size=nnz) * 2 - 1
    return rowptr, ocol, _f16bits(mag * sgn)


def random_quantized(mode: int, rows: int, cols: int, bits: int, rate: float, seed: int,
                     placement: str = "uniform", lib_size: int = 32, group_size: int = 128) -> QuantTensors:
    """Quantised tensors drawn directly (no encoder): bell-shaped indices, ascending codebooks of
    the weights' scale, CSR outliers.  Timing and decode parity do not depend on how the values
    were fitted, only on their sizes and structure."""
    rng = np.random.default_rng(seed)
    E = 1 << bits
    a = rng.integers(0, E, size=(rows, cols), dtype=np.uint8)
    b = rng.integers(0, E, size=(rows, cols), dtype=np.uint8)
    idx = ((a.astype(np.uint16) + b + 1) >> 1).astype(np.uint8)
    idx[idx >= E] = E - 1
    rowptr, ocol, oval = random_csr(rows, cols, rate, seed + 1, placement)
    if mode == 0:
        cb = np.sort(rng.standard_normal((rows, E)) * (2.0 * SIGMA0), axis=1)
        return QuantTensors(0, rows, cols, bits, idx, _f16bits(cb), rowptr, ocol, oval, group_size)
    lib = np.sort(rng.uniform(-1.0, 1.0, size=(lib_size, E)), axis=1)
    G = cols // group_size
    gid = rng.integers(0, lib_size, size=(rows, G), dtype=np.uint8)
    gscale = rng.uniform(2.0, 4.0, size=(rows, G)) * SIGMA0
    gmid = rng.standard_normal((rows, G)) * (0.1 * SIGMA0)
    return QuantTensors(1, rows, cols, bits, idx, _f16bits(lib), rowptr, ocol, oval, group_size, lib_size,
                        gid, _f16bits(gscale), _f16bits(gmid))


def random_quantized_torch(mode: int, rows: int, cols: int, bits: int, rate: float, seed: int,
                           placement: str = "uniform", lib_size: int = 32, group_size: int = 128,
                           device="cuda", library=None) -> QuantTensors:
    """`random_quantized` drawn on a torch device (seeded torch.Generator), for benchmark-sized matrices whose
    host generation would take minutes: same recipe (bell-shaped indices, ascending codebooks at the weights'
    scale, library in [-1, 1], group scale / mid-point, CSR outliers placed 'uniform' or 'clustered'), fields as
    torch tensors on `device` (fp16 values as int16 bit patterns).  `library`: a [L, 2^N] int16 tensor to share
    between the matrices of a layer.  `to_host` brings such an object back as numpy arrays."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    E = 1 << bits
    idx = torch.empty((rows, cols), dtype=torch.uint8, device=device)
    step = max(1, (64 << 20) // cols)
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        a = torch.randint(0, E, (r1 - r0, cols), generator=g, device=device, dtype=torch.int16)
        b = torch.randint(0, E, (r1 - r0, cols), generator=g, device=device, dtype=torch.int16)
        idx[r0:r1] = torch.clamp((a + b + 1) >> 1, max=E - 1).to(torch.uint8)
    # outliers
    if rate <= 0:
        rowptr = torch.zeros(rows + 1, dtype=torch.int32, device=device)
        ocol = torch.zeros(0, dtype=torch.int32, device=device)
    elif placement == "uniform":
        counts, cs = [], []
        for r0 in range(0, rows, step):
            r1 = min(rows, r0 + step)
            m = torch.rand((r1 - r0, cols), generator=g, device=device) < rate
            counts.append(m.sum(1))
            cs.append(m.nonzero()[:, 1])
        cnt = torch.cat(counts)
        ocol = torch.cat(cs).to(torch.int32)
        rowptr = torch.zeros(rows + 1, dtype=torch.int32, device=device)
        rowptr[1:] = torch.cumsum(cnt, 0).to(torch.int32)
    elif placement == "clustered":
        n_hot = max(1, int(round(rate * cols / 0.5)))
        hot = torch.sort(torch.randperm(cols, generator=g, device=device)[:n_hot]).values
        hit = torch.rand((rows, n_hot), generator=g, device=device) < 0.5
        ocol = hot[hit.nonzero()[:, 1]].to(torch.int32)
        rowptr = torch.zeros(rows + 1, dtype=torch.int32, device=device)
        rowptr[1:] = torch.cumsum(hit.sum(1), 0).to(torch.int32)
    else:
        raise ValueError(placement)
    nnz = int(ocol.numel())
    mag = (torch.rand(nnz, generator=g, device=device) * 39.0 + 10.0) * SIGMA0
    sgn = torch.randint(0, 2, (nnz,), generator=g, device=device).to(torch.float32) * 2 - 1
    oval = (mag * sgn).to(torch.float16).view(torch.int16)
    if mode == 0:
        cb = torch.sort(torch.randn((rows, E), generator=g, device=device) * (2.0 * SIGMA0), dim=1).values
        return QuantTensors(0, rows, cols, bits, idx, cb.to(torch.float16).view(torch.int16), rowptr, ocol, oval, group_size)
    if library is None:
        lib = torch.sort(torch.rand((lib_size, E), generator=g, device=device) * 2.0 - 1.0, dim=1).values
        library = lib.to(torch.float16).view(torch.int16)
    G = cols // group_size
    gid = torch.randint(0, library.shape[0], (rows, G), generator=g, device=device, dtype=torch.int16).to(torch.uint8)
    gscale = (torch.rand((rows, G), generator=g, device=device) * 2.0 + 2.0) * SIGMA0
    gmid = torch.randn((rows, G), generator=g, device=device) * (0.1 * SIGMA0)
    return QuantTensors(1, rows, cols, bits, idx, library, rowptr, ocol, oval, group_size, int(library.shape[0]), gid,
                        gscale.to(torch.float16).view(torch.int16), gmid.to(torch.float16).view(torch.int16))


def to_host(q: QuantTensors) -> QuantTensors:
    """A QuantTensors whose fields are torch tensors -> the same with numpy arrays (fp16 bit patterns as uint16)."""
    def h(t, dt):
        if t is None:
            return None
        a = t.cpu().numpy()
        return np.ascontiguousarray(a.view(np.uint16) if dt == np.uint16 else a.astype(dt))
    return QuantTensors(q.mode, q.rows, q.cols, q.bits, h(q.idx, np.uint8), h(q.codebook, np.uint16),
                        h(q.rowptr, np.int32), h(q.ocol, np.int32), h(q.oval, np.uint16), q.group_size, q.lib_size,
                        h(q.gid, np.uint8), h(q.gscale, np.uint16), h(q.gmid, np.uint16))
