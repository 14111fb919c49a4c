"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares, and
rejects bad arguments on the host before touching a GPU."""
import ctypes as C
import os
import re

import pytest

import paper_2605_14844_b200 as xfp
from paper_2605_14844_b200 import binding, build as xbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    xbuild.build()
    return xfp.load_library()


def _declared(header):
    text = open(os.path.join(ROOT, "include", header)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return set(re.findall(r"\b(xfp_[a-z0-9_]+)\s*\(", text))


def test_exports_match_header(lib):
    declared = _declared("xfp.h")
    assert declared and declared == set(binding.EXPORTS) | {n for n in declared if hasattr(lib, n)}
    for name in declared:
        assert hasattr(lib, name), name


def test_encoder_exports_match_header(lib):
    from paper_2605_14844_b200 import quant_binding
    assert sorted(f for f in os.listdir(os.path.join(ROOT, "include")) if f.endswith(".h")) == ["xfp.h", "xfp_quant.h"]
    declared = _declared("xfp_quant.h")
    assert declared == set(quant_binding.QUANT_EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_encoder_rejects_bad_arguments_on_the_host(lib):
    from paper_2605_14844_b200 import quant_binding as qb
    qb._lib()
    a, odd, n = C.c_void_p(0x1000), C.c_void_p(0x1008), None
    sz = C.c_size_t()
    assert lib.xfp_quant_workspace_size(64, 256, C.byref(sz)) == 0 and sz.value > 0
    assert lib.xfp_quant_workspace_size(64, 200, C.byref(sz)) == 3
    assert lib.xfp_quant_workspace_size(0, 256, C.byref(sz)) == 3
    big = 1 << 30
    assert lib.xfp_quant_stats(n, 100, 0, a, a, big, n) == 1
    assert lib.xfp_quant_stats(odd, 100, 0, a, a, big, n) == 2
    assert lib.xfp_quant_stats(a, 0, 0, a, a, big, n) == 3
    assert lib.xfp_quant_stats(a, 100, 2, a, a, big, n) == 3
    assert lib.xfp_quant_stats(a, 100, 0, a, a, 8, n) == 5
    assert lib.xfp_quant_outliers(a, 100, a, 0, 4.0, 0.02, n, a, a, big, n) == 1
    assert lib.xfp_quant_outliers(a, 100, a, 3, 4.0, 0.02, a, a, a, big, n) == 3
    assert lib.xfp_quant_outliers(a, 100, a, 1, 1.5, 0.0, a, a, a, big, n) == 3          # rate > 1
    assert lib.xfp_quant_outliers(a, 1 << 30, a, 0, 4.0, 0.02, a, a, a, 4096, n) == 5
    assert lib.xfp_quant_lloyd(a, n, a, 64, 256, 7, 20, a, a, n, 0, n) == 3
    assert lib.xfp_quant_lloyd(a, n, a, 64, 200, 4, 20, a, a, n, 0, n) == 3
    assert lib.xfp_quant_lloyd(a, n, a, 64, 32768, 4, 20, a, a, n, 0, n) == 1             # long channels need the workspace
    assert lib.xfp_quant_lloyd(a, n, a, 64, 32768, 4, 20, a, a, a, 4096, n) == 5
    assert lib.xfp_quant_lloyd(a, n, a, 64, 131072, 4, 20, a, a, a, big, n) == 4          # beyond the format's 65536
    assert lib.xfp_quant_lloyd(a, odd, a, 64, 256, 4, 20, a, a, n, 0, n) == 2
    assert lib.xfp_quant_libfit_library(a, 64, 4, 0, 20, a, a, big, n) == 3
    assert lib.xfp_quant_libfit_library(a, 64, 4, 32, 20, a, a, 64, n) == 5
    assert lib.xfp_quant_libfit_assign(a, n, a, 64, 256, 4, 32, 128, a, a, n, a, a, n) == 1
    assert lib.xfp_quant_libfit_assign(a, n, a, 64, 256, 4, 32, 80, a, a, a, a, a, n) == 4      # group sizes: 64, 128, 256
    assert lib.xfp_quant_libfit_assign(a, n, a, 64, 384, 4, 32, 256, a, a, a, a, a, n) == 3     # cols % group_size
    d = _desc(mode=1, lib_size=32)
    assert lib.xfp_quant_residual(C.byref(d), a, a, a, a, n, n, n, a, a, a, 10, a, big, n) == 1   # V2a needs group data
    d0 = _desc()
    assert lib.xfp_quant_residual(C.byref(d0), a, a, a, a, n, n, n, a, n, n, 10, a, big, n) == 1
    assert lib.xfp_quant_residual(C.byref(d0), a, a, a, a, n, n, n, a, a, a, 10, a, 64, n) == 5
    assert lib.xfp_quant_cosine(C.byref(d0), a, n, a, a, n, n, n, n, n) == 1
    assert lib.xfp_quant_median(a, 0, a, a, big, n) == 3
    p = qb.XfpQuantParams(0, 0, 4.0, 0.02, 0.0, 20, 0)
    r = qb.XfpQuantResult()
    cand = (C.c_int32 * 2)(4, 3)                                                          # not ascending
    assert lib.xfp_quantize(0, a, 64, 256, C.byref(p), cand, 2, 0.96, 0, a, a, a, n, n, n, n, a, a, a, 100, a,
                            C.byref(r), a, big, n) == 3
    cand = (C.c_int32 * 1)(4)
    assert lib.xfp_quantize(1, a, 64, 256, C.byref(p), cand, 1, 0.93, 32, a, a, a, n, n, n, n, a, a, a, 100, a,
                            C.byref(r), a, big, n) == 1                                   # V2a needs its outputs
    assert lib.xfp_quantize(0, a, 64, 256, C.byref(p), cand, 1, 0.96, 0, a, a, a, n, n, n, n, a, a, a, 100, a,
                            C.byref(r), a, 128, n) == 5


def _desc(**kw):
    d = dict(mode=0, rows=64, cols=256, bits=4, group_size=128, lib_size=0, col_bits=32, nnz=0)
    d.update(kw)
    return xfp.XfpDesc(*[d[n] for n, _ in xfp.XfpDesc._fields_])


def test_packed_size_accounting(lib):
    import math
    pb, wb = xfp.xfp_packed_size(_desc(rows=4096, cols=4096, nnz=50000))
    idx_bytes = 4096 * 4096 // 2
    # indices at exactly N bits per weight, codebooks, row pointers, 4 bytes per outlier (CSR), plus the
    # transposed outlier slabs: per 32-row block (C + 1) slots of 32 words, C = mean + 4 sqrt(mean) + 8
    m = math.ceil(50000 / 4096)
    slab = (4096 // 32) * (m + 4 * math.ceil(math.sqrt(m)) + 8 + 1) * 32 * 4
    base = idx_bytes + 4096 * 16 * 2 + 4097 * 4 + 50000 * 4 + slab
    assert base <= pb <= base + 6 * 256
    p0, _ = xfp.xfp_packed_size(_desc(rows=4096, cols=4096, nnz=0))
    assert p0 <= idx_bytes + 4096 * 16 * 2 + 4097 * 4 + 6 * 256
    for bits in (2, 3, 4, 5, 6):
        pb, _ = xfp.xfp_packed_size(_desc(rows=32, cols=128, bits=bits))
        assert pb >= 32 * 128 * bits // 8
    pa, _ = xfp.xfp_packed_size(_desc(mode=1, lib_size=32, rows=3072, cols=4096, bits=3, nnz=0))
    assert pa >= 3072 * 4096 * 3 // 8 + 3072 * 32 * 5 + 32 * 8 * 2


def test_group_sizes_64_128_256_are_accepted(lib):
    """The format's group size is a parameter: 64, 128 and 256 weights per group are built; the packed size of a
    V2a blob grows with the number of metadata slots (two per super-chunk at 64, one otherwise)."""
    sizes = {}
    for g in (64, 128, 256):
        pb, wb = C.c_size_t(), C.c_size_t()
        assert lib.xfp_packed_size(C.byref(_desc(mode=1, lib_size=32, rows=64, cols=1024, group_size=g)), C.byref(pb),
                                   C.byref(wb)) == 0
        sizes[g] = pb.value
        assert lib.xfp_packed_size(C.byref(_desc(rows=64, cols=1024, group_size=g)), C.byref(pb), C.byref(wb)) == 0
    assert sizes[64] > sizes[128]
    assert sizes[256] == sizes[128]


@pytest.mark.parametrize("kw,status", [
    (dict(bits=1), 3), (dict(bits=7), 3), (dict(cols=200), 3), (dict(rows=0), 3), (dict(mode=2), 3),
    (dict(group_size=80), 4), (dict(group_size=512), 4), (dict(group_size=0), 3), (dict(group_size=64, cols=192), 3),
    (dict(group_size=256, cols=384), 3), (dict(cols=131072), 4), (dict(mode=1, lib_size=0), 3), (dict(mode=1, lib_size=300), 3),
    (dict(mode=0, lib_size=32), 3), (dict(col_bits=8), 3), (dict(nnz=-1), 3),
])
def test_bad_descriptors_are_rejected(lib, kw, status):
    pb, wb = C.c_size_t(), C.c_size_t()
    d = _desc(**kw)
    assert lib.xfp_packed_size(C.byref(d), C.byref(pb), C.byref(wb)) == status


def test_null_alignment_and_size_checks_need_no_gpu(lib):
    d = _desc(nnz=5)
    a = C.c_void_p(0x1000)      # never dereferenced: every call below must fail on the host
    odd = C.c_void_p(0x1008)
    n = None
    assert lib.xfp_pack(C.byref(d), n, a, n, n, n, a, a, a, a, 1 << 30, n, n) == 1
    assert lib.xfp_pack(C.byref(d), a, a, n, n, n, n, a, a, a, 1 << 30, n, n) == 1        # nnz > 0 needs CSR
    assert lib.xfp_pack(C.byref(d), odd, a, n, n, n, a, a, a, a, 1 << 30, n, n) == 2
    assert lib.xfp_pack(C.byref(d), a, a, n, n, n, a, a, a, a, 16, n, n) == 5
    da = _desc(mode=1, lib_size=32)
    assert lib.xfp_pack(C.byref(da), a, a, n, a, a, n, n, n, a, 1 << 30, n, n) == 1       # V2a needs group ids
    assert lib.xfp_gemv_v2(C.byref(d), n, a, 1, a, 0, a, 1 << 30, n) == 1
    assert lib.xfp_gemv_v2(C.byref(d), a, a, 0, a, 0, a, 1 << 30, n) == 3
    assert lib.xfp_gemv_v2(C.byref(d), a, a, 17, a, 0, a, 1 << 30, n) == 3
    assert lib.xfp_gemv_v2(C.byref(d), a, odd, 1, a, 0, a, 1 << 30, n) == 2
    assert lib.xfp_gemv_v2(C.byref(d), a, a, 1, a, 0, a, 8, n) == 5
    assert lib.xfp_gemv_v2a(C.byref(d), a, a, 1, a, 0, a, 1 << 30, n) == 3                # V2 blob, V2a entry
    assert lib.xfp_gemv_v2(C.byref(da), a, a, 1, a, 0, a, 1 << 30, n) == 3
    assert lib.xfp_dequant(C.byref(d), a, n, n) == 1
    assert lib.xfp_dequant(C.byref(d), a, odd, n) == 2
    assert lib.xfp_gemv_grouped(C.byref(d), 0, a, a, a, 0, a, 1 << 30, n) == 3
    assert lib.xfp_gemv_grouped(C.byref(d), 4, a, a, a, 0, a, 64, n) == 5
    da64 = _desc(mode=1, lib_size=32, rows=128)
    assert lib.xfp_gemv_grouped_epilogue(C.byref(da64), 2, a, a, a, 0, 5, n, a, 1 << 30, n) == 3     # unknown epilogue
    assert lib.xfp_gemv_grouped_epilogue(C.byref(da64), 2, a, a, a, 0, 2, n, a, 1 << 30, n) == 1     # weighted sum without weights
    da96 = _desc(mode=1, lib_size=32, rows=96)
    assert lib.xfp_gemv_grouped_epilogue(C.byref(da96), 2, a, a, a, 0, 1, n, a, 1 << 30, n) == 3     # rows = 64 * k for SiLU*up
    assert lib.xfp_gemv_grouped_epilogue(C.byref(da64), 2, a, a, a, 0, 1, n, a, 64, n) == 5
    d128 = _desc(rows=128)
    assert lib.xfp_gemv_grouped_epilogue(C.byref(d128), 2, a, a, a, 0, 1, n, a, 1 << 30, n) == 4     # V2 blobs: not built
    # prefill form: V2 only, m >= 1, its own workspace size
    wsz = C.c_size_t()
    assert lib.xfp_gemm_workspace_size(C.byref(d), 64, C.byref(wsz)) == 0 and wsz.value >= 256
    assert lib.xfp_gemm_workspace_size(C.byref(d), 0, C.byref(wsz)) == 3
    assert lib.xfp_gemm_workspace_size(C.byref(da), 64, C.byref(wsz)) == 0
    dbig = _desc(mode=1, lib_size=64, bits=6)
    assert lib.xfp_gemm_workspace_size(C.byref(dbig), 64, C.byref(wsz)) == 4               # library too large for the per-bank table
    assert lib.xfp_gemm(C.byref(d), n, a, 64, a, 0, a, 1 << 30, n) == 1
    assert lib.xfp_gemm(C.byref(d), a, odd, 64, a, 0, a, 1 << 30, n) == 2
    assert lib.xfp_gemm(C.byref(d), a, a, 64, a, 3, a, 1 << 30, n) == 3                     # unknown y type
    assert lib.xfp_gemm(C.byref(d), a, a, 64, a, 0, a, 16, n) == 5
    assert lib.xfp_gemm(C.byref(dbig), a, a, 64, a, 0, a, 1 << 30, n) == 4
    wsz2 = C.c_size_t()
    assert lib.xfp_gemm_typed_workspace_size(C.byref(d), 64, 2, C.byref(wsz2)) == 0 and wsz2.value >= wsz.value + 64 * 256 * 2
    assert lib.xfp_gemm_typed_workspace_size(C.byref(d), 64, 0, C.byref(wsz2)) == 3        # x cannot be fp32
    assert lib.xfp_gemm_typed(C.byref(d), a, a, 2, 64, a, 0, a, 64, n) == 5
    assert lib.xfp_gemm_typed(C.byref(d), a, n, 2, 64, a, 0, a, 1 << 30, n) == 1
    assert xfp.xfp_status_str(0) == "ok" and "aligned" in xfp.xfp_status_str(2)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_LIB", None)
    monkeypatch.setattr(binding, "_HERE", str(tmp_path))
    with pytest.raises(xfp.XfpError):
        binding.load_library()
