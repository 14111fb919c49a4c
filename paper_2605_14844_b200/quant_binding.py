"""Python binding of the encoder's C ABI (include/xfp_quant.h): argument marshalling only.

Every function hands device pointers of torch tensors to libxfp.so; the statistics, the selection of the
extracted weights, Lloyd, LibFit, the residual and the cosine gate all run in the library's kernels.
"""
from __future__ import annotations

import ctypes as C
from typing import Optional, Sequence

import torch

from .binding import XfpDesc, XfpError, _check, _ptr, _stream, load_library

QUANT_EXPORTS = ("xfp_quant_workspace_size", "xfp_quant_stats", "xfp_quant_outliers", "xfp_quant_lloyd",
                 "xfp_quant_libfit_library", "xfp_quant_libfit_assign", "xfp_quant_residual", "xfp_quant_cosine",
                 "xfp_quant_median", "xfp_quantize")


class XfpQuantParams(C.Structure):
    """Mirror of xfp_quant_params."""
    _fields_ = [("sigma_mode", C.c_int32), ("outlier_mode", C.c_int32), ("k_sigma", C.c_double),
                ("cap_frac", C.c_double), ("rate", C.c_double), ("lloyd_iters", C.c_int32), ("group_size", C.c_int32)]


class XfpQuantResult(C.Structure):
    """Mirror of xfp_quant_result."""
    _fields_ = [("bits", C.c_int32), ("fallback", C.c_int32), ("tried", C.c_int32), ("reserved", C.c_int32),
                ("nnz", C.c_int64), ("mu", C.c_double), ("sigma", C.c_double), ("median_cos", C.c_double)]


_DECLARED = False


def _lib():
    global _DECLARED
    lib = load_library()
    if not _DECLARED:
        vp, sz, i32, i64, f64 = C.c_void_p, C.c_size_t, C.c_int32, C.c_int64, C.c_double
        dp = C.POINTER(XfpDesc)
        lib.xfp_quant_workspace_size.argtypes = [i32, i32, C.POINTER(sz)]
        lib.xfp_quant_stats.argtypes = [vp, i64, i32, vp, vp, sz, vp]
        lib.xfp_quant_outliers.argtypes = [vp, i64, vp, i32, f64, f64, vp, vp, vp, sz, vp]
        lib.xfp_quant_lloyd.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, sz, vp]
        lib.xfp_quant_libfit_library.argtypes = [vp, i32, i32, i32, i32, vp, vp, sz, vp]
        lib.xfp_quant_libfit_assign.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp]
        lib.xfp_quant_residual.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i64, vp, sz, vp]
        lib.xfp_quant_cosine.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.xfp_quant_median.argtypes = [vp, i64, vp, vp, sz, vp]
        lib.xfp_quantize.argtypes = [i32, vp, i32, i32, C.POINTER(XfpQuantParams), C.POINTER(i32), i32, f64, i32,
                                     vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i64, vp, C.POINTER(XfpQuantResult),
                                     vp, sz, vp]
        for name in QUANT_EXPORTS:
            getattr(lib, name).restype = C.c_int
        _DECLARED = True
    return lib


def _nbytes(t: torch.Tensor) -> int:
    return t.numel() * t.element_size()


def xfp_quant_workspace_size(rows: int, cols: int) -> int:
    b = C.c_size_t()
    _check(_lib().xfp_quant_workspace_size(int(rows), int(cols), C.byref(b)), "xfp_quant_workspace_size")
    return b.value


def xfp_quant_stats(W, sigma_mode: int, mu_sigma, workspace, stream=None) -> None:
    _check(_lib().xfp_quant_stats(_ptr(W), W.numel(), int(sigma_mode), _ptr(mu_sigma), _ptr(workspace),
                                  _nbytes(workspace), _stream(stream)), "xfp_quant_stats")


def xfp_quant_outliers(W, mu_sigma, outlier_mode: int, k_or_rate: float, cap_frac: float, mask, count, workspace,
                       stream=None) -> None:
    _check(_lib().xfp_quant_outliers(_ptr(W), W.numel(), _ptr(mu_sigma), int(outlier_mode), float(k_or_rate),
                                     float(cap_frac), _ptr(mask), _ptr(count), _ptr(workspace), _nbytes(workspace),
                                     _stream(stream)), "xfp_quant_outliers")


def xfp_quant_lloyd(W, mask, mu_sigma, bits: int, iters: int, codebook, idx, workspace=None, stream=None) -> None:
    """workspace: needed only for channels longer than 16384 weights."""
    rows, cols = W.shape
    _check(_lib().xfp_quant_lloyd(_ptr(W), _ptr(mask), _ptr(mu_sigma), rows, cols, int(bits), int(iters),
                                  _ptr(codebook), _ptr(idx), _ptr(workspace),
                                  0 if workspace is None else _nbytes(workspace), _stream(stream)), "xfp_quant_lloyd")


def xfp_quant_libfit_library(codebook, rows: int, bits: int, L: int, iters: int, lib, workspace, stream=None) -> None:
    _check(_lib().xfp_quant_libfit_library(_ptr(codebook), int(rows), int(bits), int(L), int(iters), _ptr(lib),
                                           _ptr(workspace), _nbytes(workspace), _stream(stream)),
           "xfp_quant_libfit_library")


def xfp_quant_libfit_assign(W, mask, mu_sigma, bits: int, L: int, lib, idx, gid, gscale, gmid, stream=None,
                            group_size: int = 128) -> None:
    rows, cols = W.shape
    _check(_lib().xfp_quant_libfit_assign(_ptr(W), _ptr(mask), _ptr(mu_sigma), rows, cols, int(bits), int(L),
                                          int(group_size), _ptr(lib), _ptr(idx), _ptr(gid), _ptr(gscale), _ptr(gmid),
                                          _stream(stream)), "xfp_quant_libfit_assign")


def xfp_quant_residual(desc: XfpDesc, W, mask, idx, codebook, gid, gscale, gmid, out_rowptr, out_col, out_val,
                       workspace, stream=None) -> None:
    cap = 0 if out_col is None else out_col.numel()
    _check(_lib().xfp_quant_residual(C.byref(desc), _ptr(W), _ptr(mask), _ptr(idx), _ptr(codebook), _ptr(gid),
                                     _ptr(gscale), _ptr(gmid), _ptr(out_rowptr), _ptr(out_col), _ptr(out_val),
                                     int(cap), _ptr(workspace), _nbytes(workspace), _stream(stream)),
           "xfp_quant_residual")


def xfp_quant_cosine(desc: XfpDesc, W, mask, idx, codebook, gid, gscale, gmid, cos, stream=None) -> None:
    _check(_lib().xfp_quant_cosine(C.byref(desc), _ptr(W), _ptr(mask), _ptr(idx), _ptr(codebook), _ptr(gid),
                                   _ptr(gscale), _ptr(gmid), _ptr(cos), _stream(stream)), "xfp_quant_cosine")


def xfp_quant_median(v, median, workspace, stream=None) -> None:
    _check(_lib().xfp_quant_median(_ptr(v), v.numel(), _ptr(median), _ptr(workspace), _nbytes(workspace),
                                   _stream(stream)), "xfp_quant_median")


class QuantBuffers:
    """Device buffers xfp_quantize writes, sized for a rows x cols matrix (allocation only)."""

    def __init__(self, rows: int, cols: int, mode: int, max_bits: int, lib_size: int, capacity: int, device="cuda",
                 group_size: int = 128):
        G = cols // group_size
        self.group_size = group_size
        e = torch.empty
        self.rows, self.cols, self.mode, self.lib_size = rows, cols, mode, lib_size
        self.mask = e((rows, cols), dtype=torch.uint8, device=device)
        self.idx = e((rows, cols), dtype=torch.uint8, device=device)
        self.codebook = e((rows, 1 << max_bits), dtype=torch.int16, device=device)
        self.lib = e((max(lib_size, 1), 1 << max_bits), dtype=torch.int16, device=device) if mode else None
        self.gid = e((rows, G), dtype=torch.uint8, device=device) if mode else None
        self.gscale = e((rows, G), dtype=torch.int16, device=device) if mode else None
        self.gmid = e((rows, G), dtype=torch.int16, device=device) if mode else None
        self.rowptr = e(rows + 1, dtype=torch.int32, device=device)
        self.ocol = e(max(capacity, 4), dtype=torch.int32, device=device)
        self.oval = e(max(capacity, 8), dtype=torch.int16, device=device)
        self.capacity = capacity
        self.cos = e(rows, dtype=torch.float64, device=device)
        self.workspace = e(xfp_quant_workspace_size(rows, cols) + 256, dtype=torch.uint8, device=device)


def xfp_quantize(mode: int, W: torch.Tensor, params: XfpQuantParams, candidates: Sequence[int], tau: float,
                 buf: QuantBuffers, stream=None) -> XfpQuantResult:
    """Algorithm 1 on the GPU; fills `buf` and returns the host-side result record."""
    rows, cols = W.shape
    cand = (C.c_int32 * len(candidates))(*[int(c) for c in candidates])
    res = XfpQuantResult()
    _check(_lib().xfp_quantize(int(mode), _ptr(W), rows, cols, C.byref(params), cand, len(candidates), float(tau),
                               int(buf.lib_size if mode else 0), _ptr(buf.mask), _ptr(buf.idx), _ptr(buf.codebook),
                               _ptr(buf.lib), _ptr(buf.gid), _ptr(buf.gscale), _ptr(buf.gmid), _ptr(buf.rowptr),
                               _ptr(buf.ocol), _ptr(buf.oval), int(buf.capacity), _ptr(buf.cos), C.byref(res),
                               _ptr(buf.workspace), _nbytes(buf.workspace), _stream(stream)), "xfp_quantize")
    return res


def quantize_and_pack(W: torch.Tensor, mode: int, candidates: Sequence[int], tau: float,
                      params: Optional[XfpQuantParams] = None, lib_size: int = 32, stream=None):
    """Float weights [rows, cols] on the device -> (PackedMatrix, XfpQuantResult): Algorithm 1 through
    xfp_quantize, then xfp_pack, without the tensors leaving the device (allocation and marshalling only)."""
    from .binding import PackedMatrix, xfp_pack, xfp_packed_size
    if params is None:
        params = XfpQuantParams(0, 0, 4.0, 0.02, 0.0, 20, 0)      # the paper's defaults: k = 4, cap 2 %, 20 rounds
    rows, cols = W.shape
    frac = params.rate if params.outlier_mode else params.cap_frac
    group = params.group_size or 128
    buf = QuantBuffers(rows, cols, mode, max(candidates), lib_size, int(frac * rows * cols), device=W.device,
                       group_size=group)
    res = xfp_quantize(mode, W, params, candidates, tau, buf, stream)
    E = 1 << res.bits
    desc = XfpDesc(mode, rows, cols, res.bits, group, lib_size if mode else 0, 32, int(res.nnz))
    pb, wb = xfp_packed_size(desc)
    packed = torch.empty(pb, dtype=torch.uint8, device=W.device)
    workspace = torch.zeros(max(wb, 16), dtype=torch.uint8, device=W.device)
    err = torch.zeros(1, dtype=torch.int32, device=W.device)
    table = (buf.lib.view(-1)[:lib_size * E] if mode else buf.codebook.view(-1)[:rows * E]).contiguous()
    xfp_pack(desc, buf.idx, table, buf.gid, buf.gscale, buf.gmid, buf.rowptr, buf.ocol, buf.oval, packed, err, stream)
    return PackedMatrix(desc, packed, workspace, err), res


def _pack_buffers(buf: QuantBuffers, mode: int, bits: int, lib_size: int, nnz: int, table: torch.Tensor, stream=None):
    """xfp_pack on the tensors an encoder call left in `buf` (allocation and marshalling only)."""
    from .binding import PackedMatrix, xfp_pack, xfp_packed_size
    desc = XfpDesc(mode, buf.rows, buf.cols, bits, buf.group_size, lib_size if mode else 0, 32, int(nnz))
    pb, wb = xfp_packed_size(desc)
    dev = buf.idx.device
    packed = torch.empty(pb, dtype=torch.uint8, device=dev)
    workspace = torch.zeros(max(wb, 16), dtype=torch.uint8, device=dev)
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    xfp_pack(desc, buf.idx, table, buf.gid, buf.gscale, buf.gmid, buf.rowptr, buf.ocol, buf.oval, packed, err, stream)
    return PackedMatrix(desc, packed, workspace, err)


def quantize_with_library(W: torch.Tensor, bits: int, lib: torch.Tensor, params: XfpQuantParams, buf: QuantBuffers,
                          stream=None) -> int:
    """V2a encoding of one matrix against a GIVEN library (the experts of a routed layer share one, "V2a: Shared
    Codebook Library"): statistics, outlier extraction, the group assignment of LibFit and the residual, each a
    library call; fills `buf` (mode 1) and returns the number of extracted weights.  lib: [L, 2^bits] int16, contiguous."""
    rows, cols = W.shape
    L = lib.shape[0]
    ms = torch.empty(2, dtype=torch.float64, device=W.device)
    count = torch.zeros(1, dtype=torch.int64, device=W.device)
    xfp_quant_stats(W, params.sigma_mode, ms, buf.workspace, stream)
    xfp_quant_outliers(W, ms, params.outlier_mode, params.rate if params.outlier_mode else params.k_sigma,
                       params.cap_frac, buf.mask, count, buf.workspace, stream)
    xfp_quant_libfit_assign(W, buf.mask, ms, bits, L, lib, buf.idx, buf.gid, buf.gscale, buf.gmid, stream,
                            group_size=buf.group_size)
    nnz = int(count.item())          # one read-back, as in xfp_quantize: the outlier arrays must hold them all
    if nnz > buf.capacity:
        raise XfpError(f"quantize_with_library: {nnz} extracted weights, buffers hold {buf.capacity}")
    desc = XfpDesc(1, rows, cols, bits, buf.group_size, L, 32, nnz)
    xfp_quant_residual(desc, W, buf.mask, buf.idx, lib, buf.gid, buf.gscale, buf.gmid, buf.rowptr, buf.ocol, buf.oval,
                       buf.workspace, stream)
    return nnz


def quantize_moe_layer(experts: Sequence[torch.Tensor], mode: int, candidates: Sequence[int] = (2, 4), tau: float = 0.93,
                       sample: Sequence[int] = (0, 1, 2, 3), params: Optional[XfpQuantParams] = None,
                       lib_size: int = 32, stream=None):
    """MoE sampling ("Auto-Selection"): Algorithm 1 once per routed layer on the stacked rows of the experts in
    `sample` (four in the paper), then every expert of the layer encoded on its own at the returned bit width --
    V2: its own per-channel codebooks; V2a: group assignments against the one library the sample's LibFit pass
    produced.  experts: float32 [rows, cols] tensors on one device.  Returns ([PackedMatrix per expert],
    XfpQuantResult of the sample, the library as an int16 tensor or None).  Every step runs in the library's kernels."""
    if params is None:
        params = XfpQuantParams(0, 0, 4.0, 0.02, 0.0, 20, 0)
    frac = params.rate if params.outlier_mode else params.cap_frac
    stacked = torch.cat([experts[i] for i in sample], dim=0).contiguous()
    rows_s, cols = stacked.shape
    group = params.group_size or 128
    sbuf = QuantBuffers(rows_s, cols, mode, max(candidates), lib_size, int(frac * rows_s * cols), device=stacked.device,
                        group_size=group)
    res = xfp_quantize(mode, stacked, params, candidates, tau, sbuf, stream)
    bits, E = int(res.bits), 1 << int(res.bits)
    lib = sbuf.lib.view(-1)[:lib_size * E].clone().view(lib_size, E) if mode else None
    out = []
    for W in experts:
        rows = W.shape[0]
        buf = QuantBuffers(rows, cols, mode, bits, lib_size, int(frac * rows * cols), device=W.device, group_size=group)
        if mode:
            nnz = quantize_with_library(W, bits, lib, params, buf, stream)
            out.append(_pack_buffers(buf, 1, bits, lib_size, nnz, lib.view(-1), stream))
        else:
            r = xfp_quantize(0, W, params, (bits,), tau, buf, stream)
            out.append(_pack_buffers(buf, 0, bits, 0, int(r.nnz), buf.codebook.view(-1)[:rows * E].contiguous(), stream))
    return out, res, lib
