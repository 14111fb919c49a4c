"""Tensor-parallel row split of an XFP linear layer (the paper deploys its models at TP = 2, "Setup").

Output channels are independent units of the fused decode GEMV, so a layer shards by rows with no change to the
kernels: rank r packs and keeps the rows [row0, row1) of the matrix -- their indices, their codebooks (V2) or their
group metadata plus the whole library (V2a), and their CSR rows -- and computes its slice of y with the same
xfp_gemv call; one all-gather of y completes the layer.  The collective is NCCL's (torch.distributed): every rank's
slice lands in local memory before anything reads it, and no kernel of this library touches a peer's memory.

Shards are cut at multiples of 32 rows (the row-block of the device layout) and have one common padded length so
that the all-gather is a single equal-sized collective; the padding of the last shard is dropped after the gather.
A split along K (each rank a slice of the indices and of x, all-reduce of y) is the other way to shard; it changes
the summation order with the rank count, so the row split, which keeps every output bit-identical to the
single-GPU result, is the one built.
"""
from __future__ import annotations

from dataclasses import replace
from typing import List, Optional, Tuple

import numpy as np


def row_partition(rows: int, world: int) -> Tuple[int, List[Tuple[int, int]]]:
    """(padded rows per rank, [(row0, row1) per rank]): contiguous slices cut at multiples of 32 rows, as even as
    the row-blocks allow; trailing ranks may own fewer rows, down to none."""
    if rows < 1 or world < 1:
        raise ValueError("rows and world must be positive")
    blocks = (rows + 31) // 32
    per = (blocks + world - 1) // world * 32
    parts = []
    for r in range(world):
        r0 = min(rows, r * per)
        parts.append((r0, min(rows, r0 + per)))
    return per, parts


def shard_tensors(q, rank: int, world: int):
    """The rows of the unpacked tensors `q` (fields of synth.QuantTensors, numpy) that `rank` owns, as an object of the
    same type; None when the rank owns no rows.  V2a shards keep the whole library."""
    _, parts = row_partition(q.rows, world)
    r0, r1 = parts[rank]
    if r1 <= r0:
        return None
    p0, p1 = int(q.rowptr[r0]), int(q.rowptr[r1])
    rowptr = (np.asarray(q.rowptr[r0:r1 + 1], dtype=np.int64) - p0).astype(np.int32)
    return replace(q, rows=r1 - r0, idx=np.ascontiguousarray(q.idx[r0:r1]),
                   codebook=q.codebook if q.mode else np.ascontiguousarray(q.codebook[r0:r1]),
                   rowptr=rowptr, ocol=np.ascontiguousarray(q.ocol[p0:p1]), oval=np.ascontiguousarray(q.oval[p0:p1]),
                   gid=None if q.gid is None else np.ascontiguousarray(q.gid[r0:r1]),
                   gscale=None if q.gscale is None else np.ascontiguousarray(q.gscale[r0:r1]),
                   gmid=None if q.gmid is None else np.ascontiguousarray(q.gmid[r0:r1]))


def gather_rows(local: np.ndarray, rows: int, world: int, dist=None) -> np.ndarray:
    """Host-side form of the all-gather (numpy, any backend): `local` is this rank's [batch, padded rows per rank]
    slice of y; returns y [batch, rows]."""
    import torch
    per, _ = row_partition(rows, world)
    t = torch.from_numpy(np.ascontiguousarray(local))
    assert t.shape[-1] == per
    if dist is None or not dist.is_initialized() or world == 1:
        return local[..., :rows]
    out = [torch.empty_like(t) for _ in range(world)]
    dist.all_gather(out, t)
    return torch.cat(out, dim=-1)[..., :rows].numpy()


class TpLinear:
    """One XFP linear layer sharded by rows over the ranks of a torch.distributed process group.

    Every rank calls `gemv(x)` with the same x [batch, cols] (fp16, on its device) and receives the whole
    y [batch, rows]: the local slice comes from the fused GEMV on the rank's shard, the rest from one all-gather."""

    def __init__(self, q, device, group=None, col_bits: int = 16):
        import torch
        import torch.distributed as dist
        from . import binding as xb
        self.dist, self.group = dist, group
        init = dist.is_available() and dist.is_initialized()
        self.world = dist.get_world_size(group) if init else 1
        self.rank = dist.get_rank(group) if init else 0
        self.rows, self.cols = q.rows, q.cols
        self.per, self.parts = row_partition(q.rows, self.world)
        shard = shard_tensors(q, self.rank, self.world)
        self.pm = xb.pack_tensors(shard, device=device, col_bits=col_bits) if shard is not None else None
        self.device = device
        self._torch = torch

    def gemv(self, x, y_fp16: bool = True, stream=None):
        torch = self._torch
        batch = x.shape[0] if x.dim() == 2 else 1
        dt = torch.float16 if y_fp16 else torch.float32
        local = torch.zeros((batch, self.per), dtype=dt, device=self.device)
        if self.pm is not None:
            r0, r1 = self.parts[self.rank]
            if batch == 1:
                self.pm.gemv(x, y=local[:, :r1 - r0], y_fp16=y_fp16, stream=stream)   # a row of y is contiguous
            else:
                local[:, :r1 - r0] = self.pm.gemv(x, y_fp16=y_fp16, stream=stream)
        if self.world == 1:
            return local[:, :self.rows]
        # [world][batch][per] after the gather: rank-major; the caller wants [batch][rows]
        full = torch.empty((self.world, batch, self.per), dtype=dt, device=self.device)
        self.dist.all_gather_into_tensor(full, local, group=self.group)
        return full.permute(1, 0, 2).reshape(batch, self.world * self.per)[:, :self.rows]
