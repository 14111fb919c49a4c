"""Python binding of the XFP C ABI (include/xfp.h): argument marshalling only.

Every function takes torch tensors (device memory, streams) and hands raw pointers to
libxfp.so; all arithmetic runs in the library's CUDA kernels.  There is no CPU fallback: if the
library has not been built the import of a function fails with XfpError.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None

EXPORTS = ("xfp_packed_size", "xfp_pack", "xfp_gemv_v2", "xfp_gemv_v2a", "xfp_gemv_grouped", "xfp_gemv_host",
           "xfp_dequant", "xfp_status_str", "xfp_gemv_v2_noalloc", "xfp_gemv_grouped_epilogue", "xfp_gemv_typed",
           "xfp_gemv_grouped_typed", "xfp_gemm", "xfp_gemm_workspace_size", "xfp_gemm_typed",
           "xfp_gemm_typed_workspace_size")

XFP_EPI_NONE, XFP_EPI_SWIGLU, XFP_EPI_COMBINE = 0, 1, 2
XFP_T_F32, XFP_T_F16, XFP_T_BF16 = 0, 1, 2


class XfpError(RuntimeError):
    pass


class XfpDesc(C.Structure):
    """Mirror of xfp_desc."""
    _fields_ = [("mode", C.c_int32), ("rows", C.c_int32), ("cols", C.c_int32), ("bits", C.c_int32),
                ("group_size", C.c_int32), ("lib_size", C.c_int32), ("col_bits", C.c_int32), ("nnz", C.c_int64)]

    def __repr__(self):
        return "XfpDesc(" + ", ".join(f"{n}={getattr(self, n)}" for n, _ in self._fields_) + ")"


def library_path() -> str:
    """libxfp.so beside this file; XFP_LIBRARY names another build of it (see build.py, XFP_LIBTAG)."""
    return os.environ.get("XFP_LIBRARY") or os.path.join(_HERE, "libxfp.so")


def load_library() -> C.CDLL:
    """dlopen libxfp.so (built in-tree by paper_2605_14844_b200/build.py) and declare its signatures."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise XfpError(f"{path} is missing: run `python -m paper_2605_14844_b200.build` (there is no fallback)")
    lib = C.CDLL(path)
    vp, sz, i32 = C.c_void_p, C.c_size_t, C.c_int32
    dp = C.POINTER(XfpDesc)
    lib.xfp_packed_size.argtypes = [dp, C.POINTER(sz), C.POINTER(sz)]
    lib.xfp_pack.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
    lib.xfp_gemv_v2.argtypes = [dp, vp, vp, i32, vp, i32, vp, sz, vp]
    lib.xfp_gemv_v2a.argtypes = [dp, vp, vp, i32, vp, i32, vp, sz, vp]
    lib.xfp_gemv_grouped.argtypes = [dp, i32, vp, vp, vp, i32, vp, sz, vp]
    lib.xfp_gemv_grouped_typed.argtypes = [dp, i32, vp, vp, i32, vp, i32, i32, vp, vp, sz, vp]
    lib.xfp_gemv_typed.argtypes = [dp, vp, vp, i32, i32, vp, i32, vp, sz, vp]
    lib.xfp_gemv_grouped_epilogue.argtypes = [dp, i32, vp, vp, vp, i32, i32, vp, vp, sz, vp]
    lib.xfp_gemv_host.argtypes = [dp, vp, vp, vp, i32, vp, vp, i32, vp, sz, vp]
    lib.xfp_dequant.argtypes = [dp, vp, vp, vp]
    lib.xfp_gemm_workspace_size.argtypes = [dp, i32, C.POINTER(sz)]
    lib.xfp_gemm.argtypes = [dp, vp, vp, i32, vp, i32, vp, sz, vp]
    lib.xfp_gemm_typed_workspace_size.argtypes = [dp, i32, i32, C.POINTER(sz)]
    lib.xfp_gemm_typed.argtypes = [dp, vp, vp, i32, i32, vp, i32, vp, sz, vp]
    lib.xfp_gemv_v2_noalloc.argtypes = [dp, vp, vp, i32, vp, i32, vp]
    lib.xfp_status_str.argtypes = [C.c_int]
    lib.xfp_status_str.restype = C.c_char_p
    for name in EXPORTS:
        if name != "xfp_status_str":
            getattr(lib, name).restype = C.c_int
    _LIB = lib
    return lib


def xfp_status_str(status: int) -> str:
    return load_library().xfp_status_str(int(status)).decode()


def _check(status: int, what: str) -> None:
    if status != 0:
        raise XfpError(f"{what}: status {status} ({xfp_status_str(status)})")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def xfp_packed_size(desc: XfpDesc):
    """(packed_bytes, workspace_bytes) for a descriptor; host-only call."""
    pb, wb = C.c_size_t(), C.c_size_t()
    _check(load_library().xfp_packed_size(C.byref(desc), C.byref(pb), C.byref(wb)), "xfp_packed_size")
    return pb.value, wb.value


def xfp_pack(desc: XfpDesc, idx, codebook, group_id, group_scale, group_mid, out_rowptr, out_col, out_val,
             packed: torch.Tensor, err_word: Optional[torch.Tensor] = None, stream=None) -> None:
    _check(load_library().xfp_pack(C.byref(desc), _ptr(idx), _ptr(codebook), _ptr(group_id), _ptr(group_scale),
                                   _ptr(group_mid), _ptr(out_rowptr), _ptr(out_col), _ptr(out_val), _ptr(packed),
                                   packed.numel() * packed.element_size(), _ptr(err_word), _stream(stream)),
           "xfp_pack")


def _gemv(fn, desc, packed, x, batch, y, y_is_fp16, workspace, stream):
    _check(fn(C.byref(desc), _ptr(packed), _ptr(x), int(batch), _ptr(y), int(bool(y_is_fp16)), _ptr(workspace),
              workspace.numel() * workspace.element_size(), _stream(stream)), fn.__name__)


def xfp_gemv_v2(desc, packed, x, batch, y, y_is_fp16, workspace, stream=None) -> None:
    _gemv(load_library().xfp_gemv_v2, desc, packed, x, batch, y, y_is_fp16, workspace, stream)


def xfp_gemv_v2a(desc, packed, x, batch, y, y_is_fp16, workspace, stream=None) -> None:
    _gemv(load_library().xfp_gemv_v2a, desc, packed, x, batch, y, y_is_fp16, workspace, stream)


_TORCH_TYPE = {torch.float32: XFP_T_F32, torch.float16: XFP_T_F16, torch.bfloat16: XFP_T_BF16}


def xfp_gemv_typed(desc, packed, x: torch.Tensor, batch, y: torch.Tensor, workspace, stream=None) -> None:
    """The fused GEMV of desc.mode with x in fp16 or bf16 and y in fp32, fp16 or bf16 (taken from the tensors' dtypes)."""
    _check(load_library().xfp_gemv_typed(C.byref(desc), _ptr(packed), _ptr(x), _TORCH_TYPE[x.dtype], int(batch), _ptr(y),
                                         _TORCH_TYPE[y.dtype], _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _stream(stream)), "xfp_gemv_typed")


def xfp_gemm_workspace_size(desc, m: int) -> int:
    b = C.c_size_t()
    _check(load_library().xfp_gemm_workspace_size(C.byref(desc), int(m), C.byref(b)), "xfp_gemm_workspace_size")
    return b.value


def xfp_gemm(desc, packed, x: torch.Tensor, y: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
    """Prefill form: y[m][rows] = x[m][cols] (D + S)^T on the tcgen05 tensor cores; x fp16, y fp32, fp16 or bf16;
    workspace: zero-filled uint8 tensor of xfp_gemm_workspace_size(desc, m) bytes (word 0 = the kernel's error flag)."""
    _check(load_library().xfp_gemm(C.byref(desc), _ptr(packed), _ptr(x), int(x.shape[0]), _ptr(y), _TORCH_TYPE[y.dtype],
                                   _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "xfp_gemm")


def xfp_gemm_typed_workspace_size(desc, m: int, x_dtype=torch.bfloat16) -> int:
    b = C.c_size_t()
    _check(load_library().xfp_gemm_typed_workspace_size(C.byref(desc), int(m), _TORCH_TYPE[x_dtype], C.byref(b)),
           "xfp_gemm_typed_workspace_size")
    return b.value


def xfp_gemm_typed(desc, packed, x: torch.Tensor, y: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
    """xfp_gemm with x in fp16 or bf16 (taken from the tensor's dtype); workspace sized by
    xfp_gemm_typed_workspace_size(desc, m, x.dtype)."""
    _check(load_library().xfp_gemm_typed(C.byref(desc), _ptr(packed), _ptr(x), _TORCH_TYPE[x.dtype], int(x.shape[0]),
                                         _ptr(y), _TORCH_TYPE[y.dtype], _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _stream(stream)), "xfp_gemm_typed")


def xfp_gemv_grouped(desc, n: int, packed_ptrs: torch.Tensor, x_ptrs: torch.Tensor, y_ptrs: torch.Tensor,
                     y_is_fp16, workspace: torch.Tensor, stream=None) -> None:
    """packed_ptrs / x_ptrs / y_ptrs: int64 device tensors holding n device addresses each."""
    _check(load_library().xfp_gemv_grouped(C.byref(desc), int(n), _ptr(packed_ptrs), _ptr(x_ptrs), _ptr(y_ptrs),
                                           int(bool(y_is_fp16)), _ptr(workspace),
                                           workspace.numel() * workspace.element_size(), _stream(stream)),
           "xfp_gemv_grouped")


def xfp_gemv_grouped_epilogue(desc, n: int, packed_ptrs: torch.Tensor, x_ptrs: torch.Tensor, y_ptrs: torch.Tensor,
                              y_is_fp16, epilogue: int, weights: Optional[torch.Tensor], workspace: torch.Tensor,
                              stream=None) -> None:
    """xfp_gemv_grouped with a fused store: XFP_EPI_SWIGLU (y[j] gets rows/2 values SiLU(gate)*up) or
    XFP_EPI_COMBINE (y[0] = sum_j weights[j] * W_j x[j]; weights: float32 device tensor of n values)."""
    _check(load_library().xfp_gemv_grouped_epilogue(C.byref(desc), int(n), _ptr(packed_ptrs), _ptr(x_ptrs),
                                                    _ptr(y_ptrs), int(bool(y_is_fp16)), int(epilogue), _ptr(weights),
                                                    _ptr(workspace), workspace.numel() * workspace.element_size(),
                                                    _stream(stream)), "xfp_gemv_grouped_epilogue")


def xfp_gemv_grouped_typed(desc, n: int, packed_ptrs: torch.Tensor, x_ptrs: torch.Tensor, x_dtype, y_ptrs: torch.Tensor,
                           y_dtype, epilogue: int, weights: Optional[torch.Tensor], workspace: torch.Tensor,
                           stream=None) -> None:
    """The grouped launch with fp16 / bf16 activations and fp32 / fp16 / bf16 outputs (torch dtypes) and an optional
    fused store (XFP_EPI_*)."""
    _check(load_library().xfp_gemv_grouped_typed(C.byref(desc), int(n), _ptr(packed_ptrs), _ptr(x_ptrs),
                                                 _TORCH_TYPE[x_dtype], _ptr(y_ptrs), _TORCH_TYPE[y_dtype], int(epilogue),
                                                 _ptr(weights), _ptr(workspace),
                                                 workspace.numel() * workspace.element_size(), _stream(stream)),
           "xfp_gemv_grouped_typed")


def xfp_gemv_host(desc, packed, x_host: torch.Tensor, x_dev, batch, y_host: torch.Tensor, y_dev, y_is_fp16,
                  workspace, stream=None) -> None:
    _check(load_library().xfp_gemv_host(C.byref(desc), _ptr(packed), _ptr(x_host), _ptr(x_dev), int(batch),
                                        _ptr(y_host), _ptr(y_dev), int(bool(y_is_fp16)), _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), _stream(stream)),
           "xfp_gemv_host")


def xfp_gemv_v2_noalloc(desc, packed, x, batch, y, y_is_fp16, stream=None) -> None:
    """V2 GEMV that uses the library's built-in 8 MiB scratch instead of a caller workspace: for callers
    that are not allowed to allocate device memory.  Calls must not overlap on the GPU (shared scratch)."""
    _check(load_library().xfp_gemv_v2_noalloc(C.byref(desc), _ptr(packed), _ptr(x), int(batch), _ptr(y),
                                              int(bool(y_is_fp16)), _stream(stream)), "xfp_gemv_v2_noalloc")


def xfp_dequant(desc, packed, W: torch.Tensor, stream=None) -> None:
    _check(load_library().xfp_dequant(C.byref(desc), _ptr(packed), _ptr(W), _stream(stream)), "xfp_dequant")


# ------------------------------------------------------------------ conveniences (still marshalling only)

def _dev(a, dtype, device):
    import numpy as np
    if a is None:
        return None
    if isinstance(a, torch.Tensor):
        return a.to(device=device).contiguous() if a.numel() else torch.zeros(16, dtype=a.dtype, device=device)
    a = np.ascontiguousarray(a)
    if a.size == 0:
        return torch.zeros(16, dtype=dtype, device=device)
    t = torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a)
    return t.to(device)


class PackedMatrix:
    """A packed blob with its descriptor and workspace (device tensors)."""

    def __init__(self, desc: XfpDesc, packed: torch.Tensor, workspace: torch.Tensor, err_word: torch.Tensor):
        self.desc, self.packed, self.workspace, self.err_word = desc, packed, workspace, err_word

    @property
    def rows(self):
        return self.desc.rows

    @property
    def cols(self):
        return self.desc.cols

    def gemv(self, x: torch.Tensor, y: Optional[torch.Tensor] = None, y_fp16: bool = False, stream=None):
        """x: fp16 [batch, cols] on the device -> y [batch, rows] fp32 (or fp16)."""
        batch = x.shape[0] if x.dim() == 2 else 1
        if y is None:
            y = torch.empty((batch, self.desc.rows), dtype=torch.float16 if y_fp16 else torch.float32, device=x.device)
        fn = xfp_gemv_v2a if self.desc.mode else xfp_gemv_v2
        fn(self.desc, self.packed, x, batch, y, y_fp16, self.workspace, stream)
        return y

    def dequant(self, stream=None) -> torch.Tensor:
        W = torch.empty((self.desc.rows, self.desc.cols), dtype=torch.float16, device=self.packed.device)
        xfp_dequant(self.desc, self.packed, W, stream)
        return W


def pack_tensors(q, device="cuda", col_bits: int = 32, stream=None) -> PackedMatrix:
    """Upload unpacked XFP tensors (any object with the fields of synth.QuantTensors) and run xfp_pack."""
    import numpy as np
    nnz = int(q.rowptr[-1])
    desc = XfpDesc(q.mode, q.rows, q.cols, q.bits, q.group_size, q.lib_size if q.mode else 0, col_bits, nnz)
    pb, wb = xfp_packed_size(desc)
    idx = _dev(q.idx, torch.uint8, device)
    cb = _dev(q.codebook, torch.int16, device)
    gid = _dev(q.gid, torch.uint8, device) if q.mode else None
    gs = _dev(q.gscale, torch.int16, device) if q.mode else None
    gm = _dev(q.gmid, torch.int16, device) if q.mode else None
    rowptr = _dev(q.rowptr, torch.int32, device)
    if isinstance(q.ocol, torch.Tensor):
        ocol = q.ocol.to(device=device, dtype=torch.int16 if col_bits == 16 else torch.int32)
        if ocol.numel() == 0:
            ocol = torch.zeros(16, dtype=ocol.dtype, device=device)
    else:
        ocol = q.ocol.astype(np.uint16) if col_bits == 16 else q.ocol.astype(np.int32)
        ocol = _dev(ocol, torch.int16 if col_bits == 16 else torch.int32, device)
    oval = _dev(q.oval, torch.int16, device)
    packed = torch.empty(pb, dtype=torch.uint8, device=device)
    workspace = torch.zeros(max(wb, 16), dtype=torch.uint8, device=device)
    err = torch.zeros(1, dtype=torch.int32, device=device)
    xfp_pack(desc, idx, cb, gid, gs, gm, rowptr, ocol, oval, packed, err, stream)
    return PackedMatrix(desc, packed, workspace, err)
