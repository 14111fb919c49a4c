"""Parity of the prefill form (xfp_gemm, tcgen05 tensor cores) against the CPU oracle, through the C ABI.

Every row of x is one GEMV of the oracle: |y_ti - y_ref_ti| <= 1e-3 * sum_k |W_ik x_tk|.  The kernel's products are
exact and its sums fp32, so it is also held far more tightly to the matrix it multiplies: up to 128 rows of x that is
D16 + S itself where the outliers are a sparse product added to the accumulator (few rows of x and few outliers),
else the dequantised matrix W^ = fp16(D16 + S) (the outliers are added to the decoded tile); both are built from the
oracle's dequantised matrices.
"""
import os

import numpy as np
import pytest
import torch

from conftest import to_oracle
from oracle import xfp_oracle as xo
import paper_2605_14844_b200 as xfp
from paper_2605_14844_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-3
TIGHT = 2e-5     # fp32 accumulation of K <= 65536 exact products, relative to sum_k |W^_ik x_tk|


def _run(q, pm, x16, dtype=torch.float32):
    xd = torch.from_numpy(x16.view(np.int16)).cuda().view(torch.float16)
    m = x16.shape[0]
    ws = torch.zeros(xfp.xfp_gemm_workspace_size(pm.desc, m), dtype=torch.uint8, device="cuda")
    y = torch.full((m, q.rows), float("nan"), dtype=dtype, device="cuda")
    xfp.xfp_gemm(pm.desc, pm.packed, xd, y, ws)
    torch.cuda.synchronize()
    words = ws[: (ws.numel() // 4) * 4].view(torch.int32)
    assert int(words[0].item()) == 0, "a bounded wait ran out in the kernel"
    n_ctrl = min(words.numel(), 1 + ((q.rows + 127) // 128) * ((m + 255) // 256))   # at least this many counters
    assert int(words[:n_ctrl].abs().sum().item()) == 0, "slice counters not left at zero"
    return y, ws, xd


def _sparse_product(pm, m):
    """Whether xfp_gemm adds the outliers as a sparse product (few rows of x, few outliers), read off the workspace it
    asks for: the transposed copy of x is the only part of it that depends on the outlier count."""
    d = pm.desc
    bare = xfp.XfpDesc(d.mode, d.rows, d.cols, d.bits, d.group_size, d.lib_size, d.col_bits, 0)
    return xfp.xfp_gemm_workspace_size(d, m) > xfp.xfp_gemm_workspace_size(bare, m)


def _check(q, pm, x16, dtype=torch.float32):
    y, _, _ = _run(q, pm, x16, dtype)
    got = y.float().cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got))
    mo = to_oracle(q)
    ref, absum = xo.gemv(mo, x16)
    err = np.abs(got - ref)
    # a bf16 store rounds the sum to 8 significant bits: half an ulp of the result on top of the GEMV bound
    tol = TOL * absum + (2.0 ** -8 * np.abs(ref) if dtype == torch.bfloat16 else 0.0) + 1e-30
    assert np.all(err <= tol), float((err / tol).max())
    if dtype == torch.float32:
        xf = x16.view(np.float16).astype(np.float64)
        if _sparse_product(pm, x16.shape[0]):
            # D16 (the dequantised matrix of the blob without its outliers) + S, exactly
            bare = xo.QuantizedMatrix(mo.mode, mo.rows, mo.cols, mo.bits, mo.idx, mo.codebook,
                                      np.zeros(mo.rows + 1, np.int32), np.zeros(0, np.int32), np.zeros(0, np.uint16),
                                      group_size=mo.group_size, lib_size=mo.lib_size, gid=mo.gid, gscale=mo.gscale,
                                      gmid=mo.gmid)
            What = xo.dequant(bare).view(np.float16).astype(np.float64)
            rows_of = np.repeat(np.arange(mo.rows), np.diff(mo.rowptr))
            np.add.at(What, (rows_of, mo.ocol), mo.oval.view(np.float16).astype(np.float64))
        else:
            What = xo.dequant(mo).view(np.float16).astype(np.float64)
        ref2 = xf @ What.T
        abs2 = np.abs(xf) @ np.abs(What).T
        err2 = np.abs(got - ref2)
        assert np.all(err2 <= TIGHT * abs2 + 1e-30), float((err2 / (abs2 + 1e-300)).max())
    return y


@pytest.mark.parametrize("mode,bits", [(0, 2), (0, 3), (0, 4), (0, 5), (0, 6), (1, 2), (1, 3), (1, 4), (1, 5)])
@pytest.mark.parametrize("m", [1, 16, 37, 128, 200])
def test_gemm_small(mode, bits, m):
    # 70 channels: one tile with a ragged row-block and a missing one; 640 columns: five super-chunks, cut along K
    q = synth.random_quantized(mode, 70, 640, bits, 0.02, seed=900 + bits + 10 * mode)
    pm = xfp.pack_tensors(q, col_bits=16 if bits % 2 else 32)
    _check(q, pm, synth.activations(m, q.cols, seed=11 + m))


@pytest.mark.parametrize("rows,cols,bits,rate", [(1, 128, 4, 0.05), (33, 128, 3, 0.0), (300, 1536, 4, 0.01),
                                                  (96, 12288, 5, 0.01), (2048, 4096, 4, 0.009), (640, 2048, 6, 0.02),
                                                  (4224, 1024, 2, 0.003)])
def test_gemm_shapes(rows, cols, bits, rate):
    q = synth.random_quantized(0, rows, cols, bits, rate, seed=rows + cols + bits)
    pm = xfp.pack_tensors(q)
    for m in (24, 130):
        _check(q, pm, synth.activations(m, cols, seed=5 + m))


@pytest.mark.parametrize("rows,cols,bits,L,rate", [(3072, 4096, 3, 32, 0.001), (4096, 1536, 3, 32, 0.001),
                                                    (300, 1536, 4, 32, 0.01), (96, 12288, 5, 32, 0.01),
                                                    (640, 2048, 2, 256, 0.02), (33, 128, 4, 1, 0.0)])
def test_gemm_v2a_shapes(rows, cols, bits, L, rate):
    """V2a: the routed experts' two projections, K slices, a ragged tile, the largest and the smallest library."""
    q = synth.random_quantized(1, rows, cols, bits, rate, seed=rows + cols + bits, lib_size=L)
    pm = xfp.pack_tensors(q)
    for m in (24, 130):
        _check(q, pm, synth.activations(m, cols, seed=7 + m))


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_gemm_output_types(dtype):
    q = synth.random_quantized(0, 200, 1024, 4, 0.01, seed=31)
    pm = xfp.pack_tensors(q)
    _check(q, pm, synth.activations(48, q.cols, seed=3), dtype)


def test_gemm_long_rows_and_spill():
    """K = 65536 (the largest the descriptor admits) and rows whose outliers overflow the slab into the CSR arrays."""
    q = synth.random_quantized(0, 40, 65536, 4, 0.005, seed=78)
    _check(q, xfp.pack_tensors(q, col_bits=16), synth.activations(20, q.cols, seed=70))
    q = synth.random_quantized(0, 64, 2048, 4, 0.01, seed=79, placement="clustered")
    _check(q, xfp.pack_tensors(q), synth.activations(20, q.cols, seed=71))


@pytest.mark.parametrize("mode,bits,placement", [(0, 4, "one_row"), (0, 3, "clustered"), (1, 4, "one_row"), (1, 2, "uniform")])
def test_gemm_outliers_as_a_sparse_product_and_in_the_tile(mode, bits, placement):
    """The two ways the kernel adds S: a sparse product in the epilogue up to 64 rows of x (here 64, with K slices, a
    ragged row-block and rows whose outliers fill the slab and spill into the CSR arrays), the scatter into the decoded
    tile beyond (65 rows); the workspace size tells which, and each is held to the matrix it multiplies."""
    q = synth.random_quantized(mode, 300, 2560, bits, 0.02, seed=1200 + bits + 10 * mode, placement=placement)
    pm = xfp.pack_tensors(q, col_bits=16)
    assert _sparse_product(pm, 64) and not _sparse_product(pm, 65)
    for m in (64, 65):
        _check(q, pm, synth.activations(m, q.cols, seed=1210 + m))
    bare = synth.random_quantized(mode, 300, 2560, bits, 0.0, seed=1230 + bits)
    pmb = xfp.pack_tensors(bare, col_bits=16)
    assert not _sparse_product(pmb, 16)
    _check(bare, pmb, synth.activations(16, bare.cols, seed=1240))


@pytest.mark.parametrize("mode,bits,m", [(0, 4, 16), (0, 3, 100), (1, 4, 48), (0, 5, 300)])
def test_gemm_more_tiles_than_sms(mode, bits, m):
    """More tiles of 128 channels than SMs: the tiered schedule -- whole tiles, one per SM, then tiles cut along K in
    halves and finer whose partial sums meet in the workspace (190 tiles on 148 SMs; 380 with two token tiles) -- held
    to the oracle on windows of channels at the start, around the boundaries of the tiers and at the ragged end; the
    counters are left zero and a second call gives the same bits."""
    rows, cols = 24250, 1024
    q = synth.random_quantized(mode, rows, cols, bits, 0.004, seed=1300 + bits + m)
    pm = xfp.pack_tensors(q, col_bits=16)
    x16 = synth.activations(m, cols, seed=1310 + m)
    y, _, _ = _run(q, pm, x16)
    y2, _, _ = _run(q, pm, x16)
    assert torch.equal(y, y2)
    got = y.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got))
    mo = to_oracle(q)
    for r0, r1 in ((0, 160), (148 * 128 - 130, 148 * 128 + 200), (21000, 21300), (rows - 290, rows)):
        ref, absum = xo.gemv(mo, x16, r0, r1)
        err = np.abs(got[:, r0:r1] - ref[:, r0:r1])
        assert np.all(err <= TOL * absum[:, r0:r1] + 1e-30), (r0, float((err / (absum[:, r0:r1] + 1e-300)).max()))


def test_gemm_matches_gemv_rows_and_is_deterministic():
    q = synth.random_quantized(0, 512, 4096, 4, 0.01, seed=41)
    pm = xfp.pack_tensors(q)
    x16 = synth.activations(64, q.cols, seed=9)
    y1, _, xd = _run(q, pm, x16)
    y2, _, _ = _run(q, pm, x16)
    assert torch.equal(y1, y2)
    # the same matrix through the decode kernel, row by row of x: both sit inside the oracle's bound, so they
    # differ by at most twice that bound
    _, absum = xo.gemv(to_oracle(q), x16[:2])
    for t in range(2):
        yv = pm.gemv(xd[t:t + 1]).float().cpu().numpy().astype(np.float64)[0]
        assert np.all(np.abs(yv - y1[t].cpu().numpy().astype(np.float64)) <= 2 * TOL * absum[t] + 1e-30)


def test_gemm_rejects():
    q = synth.random_quantized(1, 64, 256, 6, 0.0, seed=1)
    pm = xfp.pack_tensors(q)
    with pytest.raises(xfp.XfpError):
        xfp.xfp_gemm_workspace_size(pm.desc, 16)      # V2a, N = 6, L = 32: the per-bank library does not fit
    q = synth.random_quantized(0, 64, 256, 4, 0.0, seed=1)
    pm = xfp.pack_tensors(q)
    x = torch.zeros((16, 256), dtype=torch.float16, device="cuda")
    y = torch.zeros((16, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(xfp.XfpError):
        xfp.xfp_gemm(pm.desc, pm.packed, x, y, torch.zeros(16, dtype=torch.uint8, device="cuda"))   # workspace too small


def _random_case(rng):
    mode = int(rng.integers(0, 2))
    bits = int(rng.integers(2, 7 if mode == 0 else 6))
    rows = int(rng.choice([1, 31, 32, 97, 128, 129, 260, 511, 1000]))
    cols = 128 * int(rng.choice([1, 2, 3, 5, 8, 13, 24]))
    rate = float(rng.choice([0.0, 0.001, 0.01, 0.05]))
    placement = str(rng.choice(["uniform", "clustered", "one_row"]))
    m = int(rng.choice([1, 2, 15, 16, 17, 100, 128, 129, 257]))
    L = int(rng.choice([1, 7, 32])) if mode else 32
    return mode, bits, rows, cols, rate, placement, m, L


@pytest.mark.parametrize("i", range(int(os.environ.get("XFP_GEMM_SWEEP_CASES", "32"))))
def test_gemm_randomized(i):
    """Seeded random shapes, bit widths, outlier rates and placements, library sizes and numbers of rows of x."""
    rng = np.random.default_rng(int(os.environ.get("XFP_SWEEP_SEED", "2605")) * 1000 + i)
    mode, bits, rows, cols, rate, placement, m, L = _random_case(rng)
    q = synth.random_quantized(mode, rows, cols, bits, rate, seed=7000 + i, placement=placement, lib_size=L)
    pm = xfp.pack_tensors(q, col_bits=16 if i % 2 else 32)
    _check(q, pm, synth.activations(m, cols, seed=8000 + i), [torch.float32, torch.float32, torch.float16][i % 3])


@pytest.mark.parametrize("mode,bits,m", [(0, 4, 40), (0, 5, 300), (1, 3, 130), (0, 2, 1)])
def test_gemm_bf16_activations(mode, bits, m):
    """xfp_gemm_typed: bf16 rows of x (converted to fp16 by a kernel of the library, then the same GEMM); reference: the
    oracle on the exact bf16 values; tolerance: the GEMV bound plus the conversion's 2^-25 per weight for tiny |x|."""
    q = synth.random_quantized(mode, 200, 1024, bits, 0.01, seed=5100 + bits)
    pm = xfp.pack_tensors(q)
    g = torch.Generator().manual_seed(5200 + m)
    xb = torch.randn((m, q.cols), generator=g, dtype=torch.float32).to(torch.bfloat16)
    x64 = xb.to(torch.float64).numpy()
    mo = to_oracle(q)
    ref, absum = xo.gemv_x64(mo, x64)
    tiny = 2.0 ** -25 * np.abs(xo.dequant(mo).view(np.float16).astype(np.float64)).sum(1)[None, :]
    for dt, ulp in ((torch.float32, 0.0), (torch.bfloat16, 2.0 ** -8)):
        ws = torch.zeros(xfp.xfp_gemm_typed_workspace_size(pm.desc, m, torch.bfloat16), dtype=torch.uint8, device="cuda")
        y = torch.full((m, q.rows), float("nan"), dtype=dt, device="cuda")
        xfp.xfp_gemm_typed(pm.desc, pm.packed, xb.cuda(), y, ws)
        torch.cuda.synchronize()
        assert int(ws[:4].view(torch.int32).item()) == 0
        got = y.to(torch.float64).cpu().numpy()
        tol = TOL * absum + tiny + ulp * np.abs(ref) + 1e-30
        assert np.all(np.abs(got - ref) <= tol), float((np.abs(got - ref) / tol).max())
    # fp16 rows of x through the typed entry are the plain call
    x16 = synth.activations(m, q.cols, seed=5300)
    xd = torch.from_numpy(x16.view(np.int16)).cuda().view(torch.float16)
    ws = torch.zeros(xfp.xfp_gemm_typed_workspace_size(pm.desc, m, torch.float16), dtype=torch.uint8, device="cuda")
    y1 = torch.empty((m, q.rows), dtype=torch.float32, device="cuda")
    xfp.xfp_gemm_typed(pm.desc, pm.packed, xd, y1, ws)
    y2, _, _ = _run(q, pm, x16)
    assert torch.equal(y1, y2)
