"""ctypes front end of the C oracle (oracle/xfp_oracle.c) plus the encoder's driver loops.

Test infrastructure only.  Everything here is CPU, fp64 unless the format fixes fp32, and
shares no code with the CUDA library.  Section names refer to the XFP paper.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass, field
from typing import Optional, Sequence

import numpy as np

from . import build as _build

_lib = C.CDLL(_build.build())

_u8p = np.ctypeslib.ndpointer(np.uint8, flags="C_CONTIGUOUS")
_u16p = np.ctypeslib.ndpointer(np.uint16, flags="C_CONTIGUOUS")
_i32p = np.ctypeslib.ndpointer(np.int32, flags="C_CONTIGUOUS")
_f32p = np.ctypeslib.ndpointer(np.float32, flags="C_CONTIGUOUS")
_f64p = np.ctypeslib.ndpointer(np.float64, flags="C_CONTIGUOUS")


class _CMatrix(C.Structure):
    _fields_ = [("mode", C.c_int32), ("rows", C.c_int32), ("cols", C.c_int32), ("bits", C.c_int32),
                ("group_size", C.c_int32), ("lib_size", C.c_int32),
                ("idx", C.c_void_p), ("codebook", C.c_void_p), ("gid", C.c_void_p),
                ("gscale", C.c_void_p), ("gmid", C.c_void_p),
                ("rowptr", C.c_void_p), ("ocol", C.c_void_p), ("oval", C.c_void_p)]


_lib.xo_half_to_double.restype = C.c_double
_lib.xo_half_to_double.argtypes = [C.c_uint16]
_lib.xo_double_to_half.restype = C.c_uint16
_lib.xo_double_to_half.argtypes = [C.c_double]
_lib.xo_float_to_half.restype = C.c_uint16
_lib.xo_float_to_half.argtypes = [C.c_float]
_lib.xo_halfs_to_doubles.argtypes = [C.c_int64, _u16p, _f64p]
_lib.xo_doubles_to_halfs.argtypes = [C.c_int64, _f64p, _u16p]
_lib.xo_v2a_value16.restype = C.c_uint16
_lib.xo_v2a_value16.argtypes = [C.c_uint16, C.c_uint16, C.c_uint16]
_lib.xo_table1.argtypes = [C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]
_lib.xo_table1_words.restype = C.c_int64
_lib.xo_table1_words.argtypes = [C.c_int, C.c_int64]
_lib.xo_table1_pack_row.argtypes = [C.c_int, _u8p, C.c_int64, C.c_void_p]
_lib.xo_table1_unpack_row.argtypes = [C.c_int, C.c_void_p, C.c_int64, _u8p]
_lib.xo_dequant.argtypes = [C.POINTER(_CMatrix), _u16p]
_lib.xo_gemv_rows.argtypes = [C.POINTER(_CMatrix), _u16p, C.c_int32, C.c_int64, C.c_int64, _f64p, _f64p]
_lib.xo_gemv_rows_x64.argtypes = [C.POINTER(_CMatrix), _f64p, C.c_int32, C.c_int64, C.c_int64, _f64p, _f64p]
_lib.xo_threads.restype = C.c_int
_lib.xo_set_threads.argtypes = [C.c_int]
_lib.xo_stats.argtypes = [_f32p, C.c_int64, C.POINTER(C.c_double), C.POINTER(C.c_double)]
_lib.xo_robust_sigma.restype = C.c_double
_lib.xo_robust_sigma.argtypes = [_f32p, C.c_int64, C.c_double]
_lib.xo_outlier_mask.restype = C.c_int64
_lib.xo_outlier_mask.argtypes = [_f32p, C.c_int64, C.c_double, C.c_double, C.c_double, _u8p]
_lib.xo_outlier_top_rate.restype = C.c_int64
_lib.xo_outlier_top_rate.argtypes = [_f32p, C.c_int64, C.c_double, C.c_double, _u8p]
_lib.xo_lloyd_row.restype = C.c_int
_lib.xo_lloyd_row.argtypes = [_f64p, C.c_int64, C.c_int, C.c_int, _u16p, _u8p, C.c_void_p]
_lib.xo_quantize_v2.argtypes = [_f32p, C.c_int64, C.c_int64, C.c_void_p, C.c_double, C.c_int, C.c_int, _u8p, _u16p]
_lib.xo_residual.argtypes = [_f32p, _u16p, _u8p, C.c_int64, C.c_int64, _i32p, _i32p, _u16p]
_lib.xo_row_cosine.argtypes = [_f32p, _u16p, C.c_int64, C.c_int64, _f64p]
_lib.xo_libfit_library.argtypes = [_u16p, C.c_int64, C.c_int, C.c_int, C.c_int, _u16p]
_lib.xo_libfit_assign.argtypes = [_f32p, C.c_int64, C.c_int64, C.c_void_p, C.c_double, C.c_int, C.c_int, C.c_int,
                                  _u16p, _u8p, _u8p, _u16p, _u16p]

MODE_V2 = 0
MODE_V2A = 1


# ---------------------------------------------------------------- fp16

def half_to_double(h) -> np.ndarray:
    """fp16 bit patterns (uint16) -> float64, the oracle's own decoder."""
    h = np.ascontiguousarray(h, dtype=np.uint16)
    out = np.empty(h.shape, dtype=np.float64)
    _lib.xo_halfs_to_doubles(h.size, h.reshape(-1), out.reshape(-1))
    return out


def double_to_half(d) -> np.ndarray:
    """float64 -> fp16 bit patterns, round to nearest even, the oracle's own encoder."""
    d = np.ascontiguousarray(d, dtype=np.float64)
    out = np.empty(d.shape, dtype=np.uint16)
    _lib.xo_doubles_to_halfs(d.size, d.reshape(-1), out.reshape(-1))
    return out


def v2a_value16(scale: int, lib: int, mid: int) -> int:
    return int(_lib.xo_v2a_value16(scale, lib, mid))


# ---------------------------------------------------------------- Table 1

def table1(bits: int):
    """(values per word, word width in bits) of the paper's Table 1."""
    v, w = C.c_int(), C.c_int()
    if _lib.xo_table1(bits, C.byref(v), C.byref(w)):
        raise ValueError(f"no Table 1 row for N={bits}")
    return v.value, w.value


def table1_pack_row(bits: int, idx: np.ndarray) -> np.ndarray:
    idx = np.ascontiguousarray(idx, dtype=np.uint8)
    _, wb = table1(bits)
    nw = _lib.xo_table1_words(bits, idx.size)
    words = np.zeros(nw, dtype=np.uint32 if wb == 32 else np.uint16)
    _lib.xo_table1_pack_row(bits, idx, idx.size, words.ctypes.data)
    return words


def table1_unpack_row(bits: int, words: np.ndarray, cols: int) -> np.ndarray:
    out = np.empty(cols, dtype=np.uint8)
    words = np.ascontiguousarray(words)
    _lib.xo_table1_unpack_row(bits, words.ctypes.data, cols, out)
    return out


# ---------------------------------------------------------------- the quantised matrix

@dataclass
class QuantizedMatrix:
    """The unpacked XFP tensors of one linear layer (numpy, host)."""
    mode: int
    rows: int
    cols: int
    bits: int
    idx: np.ndarray                       # uint8 [rows, cols]
    codebook: np.ndarray                  # uint16 (fp16 bits): V2 [rows, 2^N]; V2a [L, 2^N]
    rowptr: np.ndarray                    # int32 [rows+1]
    ocol: np.ndarray                      # int32 [nnz]
    oval: np.ndarray                      # uint16 [nnz]
    group_size: int = 128
    lib_size: int = 0
    gid: Optional[np.ndarray] = None      # uint8 [rows, cols/group]
    gscale: Optional[np.ndarray] = None   # uint16 [rows, cols/group]
    gmid: Optional[np.ndarray] = None     # uint16 [rows, cols/group]
    info: dict = field(default_factory=dict)

    @property
    def nnz(self) -> int:
        return int(self.rowptr[-1])

    def _c(self) -> _CMatrix:
        def p(a):
            return None if a is None else a.ctypes.data
        for name, dt in (("idx", np.uint8), ("codebook", np.uint16), ("rowptr", np.int32), ("ocol", np.int32),
                         ("oval", np.uint16), ("gid", np.uint8), ("gscale", np.uint16), ("gmid", np.uint16)):
            a = getattr(self, name)
            if a is not None:
                assert a.dtype == dt and a.flags["C_CONTIGUOUS"], name
        return _CMatrix(self.mode, self.rows, self.cols, self.bits, self.group_size, self.lib_size,
                        p(self.idx), p(self.codebook), p(self.gid), p(self.gscale), p(self.gmid),
                        p(self.rowptr), p(self.ocol), p(self.oval))


def dequant(m: QuantizedMatrix) -> np.ndarray:
    """W^ = fp16(D16 + S) as fp16 bit patterns [rows, cols] (Eq. 1)."""
    out = np.empty((m.rows, m.cols), dtype=np.uint16)
    cm = m._c()
    _lib.xo_dequant(C.byref(cm), out.reshape(-1))
    return out


def gemv(m: QuantizedMatrix, x16: np.ndarray, row0: int = 0, row1: Optional[int] = None):
    """fp64 y[b, i] = sum_k (D_ik + S_ik) x[b, k] and absum[b, i] = sum_k |(D_ik + S_ik) x[b, k]|.

    x16: fp16 bit patterns [batch, cols].  Rows outside [row0, row1) are left at zero.
    """
    x16 = np.ascontiguousarray(x16, dtype=np.uint16).reshape(-1, m.cols)
    batch = x16.shape[0]
    row1 = m.rows if row1 is None else row1
    y = np.zeros((batch, m.rows), dtype=np.float64)
    a = np.zeros((batch, m.rows), dtype=np.float64)
    cm = m._c()
    _lib.xo_gemv_rows(C.byref(cm), x16.reshape(-1), batch, row0, row1, y.reshape(-1), a.reshape(-1))
    return y, a


def gemv_x64(m: QuantizedMatrix, x: np.ndarray, row0: int = 0, row1: Optional[int] = None):
    """gemv for activations given as real numbers [batch, cols] (bf16 values are exact in fp64)."""
    x = np.ascontiguousarray(x, dtype=np.float64).reshape(-1, m.cols)
    batch = x.shape[0]
    row1 = m.rows if row1 is None else row1
    y = np.zeros((batch, m.rows), dtype=np.float64)
    a = np.zeros((batch, m.rows), dtype=np.float64)
    cm = m._c()
    _lib.xo_gemv_rows_x64(C.byref(cm), x.reshape(-1), batch, row0, row1, y.reshape(-1), a.reshape(-1))
    return y, a


def threads() -> int:
    return int(_lib.xo_threads())


def set_threads(n: int) -> None:
    _lib.xo_set_threads(int(n))


# ---------------------------------------------------------------- a routed expert's feed-forward block

def silu_mul(gate: np.ndarray, up: np.ndarray) -> np.ndarray:
    """h = SiLU(gate) * up with SiLU(g) = g / (1 + exp(-g)), in fp64: the element-wise step between the
    gate_up and the down projection of a gated feed-forward block (the routed experts of the paper's MoE
    models; the fused decode path applies it in the store of the gate_up GEMV)."""
    g = np.asarray(gate, dtype=np.float64)
    return g / (1.0 + np.exp(-g)) * np.asarray(up, dtype=np.float64)


# ---------------------------------------------------------------- encoder

def stats(W: np.ndarray):
    """(mu, sigma): mean and population standard deviation of the whole matrix (Outlier Extraction)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    mu, sg = C.c_double(), C.c_double()
    _lib.xo_stats(W.reshape(-1), W.size, C.byref(mu), C.byref(sg))
    return mu.value, sg.value


def outlier_mask(W: np.ndarray, k: float = 4.0, cap: float = 0.02, sigma_mode: str = "matrix",
                 rate: Optional[float] = None):
    """Mask of extracted weights: |w - mu| > k*sigma capped at `cap` of the matrix (paper default
    k = 4, cap 2 %).  sigma_mode 'robust' uses 1.4826*median|w - mu|; `rate` instead takes exactly
    the top fraction by |w - mu| (both are conveniences for synthetic workloads, not the paper's)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    mu, sg = stats(W)
    mask = np.zeros(W.shape, dtype=np.uint8)
    if rate is not None:
        _lib.xo_outlier_top_rate(W.reshape(-1), W.size, mu, float(rate), mask.reshape(-1))
        return mask, mu, sg
    if sigma_mode == "robust":
        sg = float(_lib.xo_robust_sigma(W.reshape(-1), W.size, mu))
    elif sigma_mode != "matrix":
        raise ValueError(sigma_mode)
    _lib.xo_outlier_mask(W.reshape(-1), W.size, mu, k * sg, cap, mask.reshape(-1))
    return mask, mu, sg


def lloyd_row(v: np.ndarray, bits: int, iters: int = 20, want_trace: bool = False):
    """Per-channel Lloyd on one row of bulk values -> (codebook fp16 bits, indices, rounds[, trace])."""
    v = np.ascontiguousarray(v, dtype=np.float64)
    cb = np.empty(1 << bits, dtype=np.uint16)
    idx = np.empty(v.size, dtype=np.uint8)
    trace = np.zeros(iters + 1, dtype=np.float64) if want_trace else None
    done = _lib.xo_lloyd_row(v, v.size, bits, iters, cb, idx, None if trace is None else trace.ctypes.data)
    return (cb, idx, done, trace) if want_trace else (cb, idx, done)


def _finish(W, mask, m: QuantizedMatrix) -> QuantizedMatrix:
    """Attach the residual S = fp16(w - D16) at the extracted positions, in CSR."""
    rows, cols = W.shape
    nnz = int(mask.sum())
    m.rowptr = np.zeros(rows + 1, dtype=np.int32)
    m.ocol = np.zeros(0, dtype=np.int32)
    m.oval = np.zeros(0, dtype=np.uint16)
    D16 = dequant(m)
    rowptr = np.zeros(rows + 1, dtype=np.int32)
    ocol = np.zeros(max(nnz, 1), dtype=np.int32)
    oval = np.zeros(max(nnz, 1), dtype=np.uint16)
    _lib.xo_residual(W.reshape(-1), D16.reshape(-1), mask.reshape(-1), rows, cols, rowptr, ocol, oval)
    m.rowptr, m.ocol, m.oval = rowptr, ocol[:nnz].copy(), oval[:nnz].copy()
    return m


def quantize_v2(W: np.ndarray, bits: int, mask: np.ndarray, mu: float, iters: int = 20) -> QuantizedMatrix:
    """V2: outliers out, one Lloyd codebook per output channel, residual CSR."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    rows, cols = W.shape
    idx = np.empty((rows, cols), dtype=np.uint8)
    cb = np.empty((rows, 1 << bits), dtype=np.uint16)
    _lib.xo_quantize_v2(W.reshape(-1), rows, cols, mask.ctypes.data, mu, bits, iters, idx.reshape(-1), cb.reshape(-1))
    m = QuantizedMatrix(MODE_V2, rows, cols, bits, idx, cb, None, None, None)
    return _finish(W, mask, m)


def quantize_v2a(W: np.ndarray, bits: int, mask: np.ndarray, mu: float, lib_size: int = 32, iters: int = 20,
                 group: int = 128, library: Optional[np.ndarray] = None) -> QuantizedMatrix:
    """V2a: LibFit over the per-channel codebooks, then per-group re-indexing.

    `library` lets several matrices of a layer (experts) share one library learned elsewhere."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    rows, cols = W.shape
    E = 1 << bits
    if library is None:
        idx0 = np.empty((rows, cols), dtype=np.uint8)
        cb = np.empty((rows, E), dtype=np.uint16)
        _lib.xo_quantize_v2(W.reshape(-1), rows, cols, mask.ctypes.data, mu, bits, iters, idx0.reshape(-1), cb.reshape(-1))
        library = np.empty((lib_size, E), dtype=np.uint16)
        _lib.xo_libfit_library(cb.reshape(-1), rows, bits, lib_size, iters, library.reshape(-1))
    library = np.ascontiguousarray(library, dtype=np.uint16)
    G = cols // group
    idx = np.empty((rows, cols), dtype=np.uint8)
    gid = np.empty((rows, G), dtype=np.uint8)
    gs = np.empty((rows, G), dtype=np.uint16)
    gm = np.empty((rows, G), dtype=np.uint16)
    _lib.xo_libfit_assign(W.reshape(-1), rows, cols, mask.ctypes.data, mu, bits, library.shape[0], group,
                          library.reshape(-1), idx.reshape(-1), gid.reshape(-1), gs.reshape(-1), gm.reshape(-1))
    m = QuantizedMatrix(MODE_V2A, rows, cols, bits, idx, library, None, None, None, group_size=group,
                        lib_size=library.shape[0], gid=gid, gscale=gs, gmid=gm)
    return _finish(W, mask, m)


def row_cosine(W: np.ndarray, What16: np.ndarray) -> np.ndarray:
    """cos_i between original channel i and its reconstruction (Algorithm 1)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    out = np.empty(W.shape[0], dtype=np.float64)
    _lib.xo_row_cosine(W.reshape(-1), np.ascontiguousarray(What16).reshape(-1), W.shape[0], W.shape[1], out)
    return out


def median(v: np.ndarray) -> float:
    s = np.sort(np.asarray(v, dtype=np.float64))
    n = s.size
    return float(s[n // 2]) if n & 1 else float(0.5 * (s[n // 2 - 1] + s[n // 2]))


def auto_select(W: np.ndarray, layer_class: str = "attention", candidates: Sequence[int] = (2, 3, 4),
                tau_strict: float = 0.96, tau_lazy: float = 0.93, mode: int = MODE_V2, k: float = 4.0,
                cap: float = 0.02, sigma_mode: str = "matrix", rate: Optional[float] = None, iters: int = 20,
                lib_size: int = 32, group: int = 128) -> QuantizedMatrix:
    """Algorithm 1 (two-threshold auto-select): ascending N, first whose median per-channel cosine
    reaches the class's floor; otherwise the largest candidate (info['fallback'] = True)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    mask, mu, sg = outlier_mask(W, k=k, cap=cap, sigma_mode=sigma_mode, rate=rate)
    tau = tau_lazy if layer_class == "moe_routed" else tau_strict
    tried = []
    m = None
    for n in sorted(candidates):
        m = quantize_v2(W, n, mask, mu, iters) if mode == MODE_V2 else quantize_v2a(W, n, mask, mu, lib_size, iters, group)
        cosv = row_cosine(W, dequant(m))
        med = median(cosv)
        tried.append((n, med))
        m.info = {"tau": tau, "median_cos": med, "min_cos": float(cosv.min()), "frac_below": float((cosv < tau).mean()),
                  "fallback": False, "tried": list(tried), "mu": mu, "sigma": sg}
        if med >= tau:
            return m
    m.info["fallback"] = True
    return m


def auto_select_moe(experts: Sequence[np.ndarray], sample: Sequence[int] = (0, 1, 2, 3),
                    candidates: Sequence[int] = (2, 4), tau: float = 0.93, mode: int = MODE_V2A, k: float = 4.0,
                    cap: float = 0.02, sigma_mode: str = "matrix", rate: Optional[float] = None, iters: int = 20,
                    lib_size: int = 32):
    """MoE sampling ("Auto-Selection"): Algorithm 1 runs once per routed layer, on the rows of a few experts (four in
    the paper) stacked into one matrix, and the bit width it returns is used for every expert of the layer.

    Steps: (1) auto_select on the concatenation of experts[i], i in `sample`, with the lazy threshold `tau`;
    (2) every expert is then quantised on its own at that width -- its own mu, sigma and extracted weights, its own
    per-channel codebooks (V2) or, for V2a, group assignments against the ONE library the sample's LibFit pass
    produced, which the experts of the layer share.  Returns (list of QuantizedMatrix, the sample's info dict)."""
    mats = [np.ascontiguousarray(W, dtype=np.float32) for W in experts]
    picked = np.concatenate([mats[i] for i in sample], axis=0)
    probe = auto_select(picked, "moe_routed", candidates, tau_lazy=tau, mode=mode, k=k, cap=cap, sigma_mode=sigma_mode,
                        rate=rate, iters=iters, lib_size=lib_size)
    out = []
    for W in mats:
        mask, mu, _ = outlier_mask(W, k=k, cap=cap, sigma_mode=sigma_mode, rate=rate)
        if mode == MODE_V2:
            out.append(quantize_v2(W, probe.bits, mask, mu, iters))
        else:
            out.append(quantize_v2a(W, probe.bits, mask, mu, lib_size, iters, library=probe.codebook))
    info = dict(probe.info, bits=probe.bits, sample=tuple(int(i) for i in sample))
    return out, info
