"""xfp_gemv_v2_noalloc: the V2 GEMV for callers that may not allocate device memory (a plug-in inside an
application that owns all GPU memory, or a latency-critical path where cudaMalloc is forbidden).  It
takes no workspace: the split-K scratch lives in an 8 MiB array inside the library.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from conftest import to_oracle
from oracle import xfp_oracle as xo
import paper_2605_14844_b200 as xfp
from paper_2605_14844_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-3   # the GEMV tolerance of the parity tests: |y - y_ref| <= 1e-3 * sum_k |W_ik x_k|


def _xdev(x16):
    return torch.from_numpy(x16.view(np.int16)).cuda().view(torch.float16)


@pytest.mark.parametrize("bits,rows,cols,batch,y_fp16", [(6, 512, 4096, 1, 0), (4, 1024, 2048, 3, 0),
                                                         (4, 512, 4096, 1, 1)])
def test_noalloc_matches_the_oracle_and_the_workspace_entry_point_twice(bits, rows, cols, batch, y_fp16):
    # shapes that split K, so the scratch (partial sums and counters) is really used
    q = synth.random_quantized(0, rows, cols, bits, 0.01, seed=4242 + bits)
    pm = xfp.pack_tensors(q, col_bits=16)
    lib = xfp.load_library()
    ydt = torch.float16 if y_fp16 else torch.float32
    for call in range(2):                                   # two calls in a row share the built-in scratch
        x16 = synth.activations(batch, cols, seed=50 + call)
        x = _xdev(x16)
        y_ws = torch.zeros((batch, rows), dtype=ydt, device="cuda")
        y_na = torch.full((batch, rows), float("nan"), dtype=ydt, device="cuda")
        xfp.xfp_gemv_v2(pm.desc, pm.packed, x, batch, y_ws, bool(y_fp16), pm.workspace)
        st = lib.xfp_gemv_v2_noalloc(C.byref(pm.desc), C.c_void_p(pm.packed.data_ptr()), C.c_void_p(x.data_ptr()),
                                     batch, C.c_void_p(y_na.data_ptr()), y_fp16,
                                     C.c_void_p(torch.cuda.current_stream().cuda_stream))
        assert st == 0, xfp.xfp_status_str(st)
        torch.cuda.synchronize()
        ref, absum = xo.gemv(to_oracle(q), x16)
        got = y_na.float().cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(got))
        assert np.all(np.abs(got - ref) <= TOL * absum)                                    # against the oracle
        assert np.all(np.abs(got - y_ws.float().cpu().numpy().astype(np.float64)) <= TOL * absum)
        # the summation order is fixed and the same in both entry points: identical bits
        assert torch.equal(y_na.view(torch.int16 if y_fp16 else torch.int32),
                           y_ws.view(torch.int16 if y_fp16 else torch.int32))


def test_noalloc_rejects_shapes_beyond_the_builtin_scratch():
    lib = xfp.load_library()
    big = xfp.XfpDesc(0, 28672, 8192, 4, 128, 0, 16, 0)     # its workspace is larger than 8 MiB
    a = C.c_void_p(0x1000)                                  # never dereferenced: rejected on the host
    assert lib.xfp_gemv_v2_noalloc(C.byref(big), a, a, 1, a, 0, None) == 5
    bad = xfp.XfpDesc(0, 64, 200, 4, 128, 0, 16, 0)         # invalid descriptors are reported as such
    assert lib.xfp_gemv_v2_noalloc(C.byref(bad), a, a, 1, a, 0, None) == 3
