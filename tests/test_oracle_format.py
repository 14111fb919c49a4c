"""Pins for the oracle's format half: fp16, Table 1 packing, dequantisation and the fp64 GEMV.

Every check compares the oracle with something that is not the oracle: numpy's fp16, exact
integer/rational arithmetic, hand-worked words, closed forms, scipy's sparse matvec, or a brute
force written independently here.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.sparse as sp

from conftest import read_golden, to_oracle
from oracle import xfp_oracle as xo
from paper_2605_14844_b200 import synth


# ---------------------------------------------------------------- fp16

def test_fp16_decode_all_patterns_match_numpy():
    h = np.arange(65536, dtype=np.uint16)
    mine = xo.half_to_double(h)
    ref = h.view(np.float16).astype(np.float64)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(mine), nan)
    assert np.array_equal(mine[~nan], ref[~nan])
    assert np.array_equal(np.signbit(mine[~nan]), np.signbit(ref[~nan]))


def test_fp16_roundtrip_identity():
    h = np.arange(65536, dtype=np.uint16)
    d = xo.half_to_double(h)
    back = xo.double_to_half(d)
    ok = ~np.isnan(d)
    assert np.array_equal(back[ok], h[ok])


def test_fp16_round_to_nearest_even_at_midpoints():
    # positive finite neighbours: the midpoint must go to the pattern with an even last bit
    h = np.arange(0, 0x7bff, dtype=np.uint16)
    lo = xo.half_to_double(h)
    hi = xo.half_to_double(h + 1)
    mid = 0.5 * (lo + hi)              # exact in fp64
    got = xo.double_to_half(mid)
    want = np.where(h % 2 == 0, h, h + 1).astype(np.uint16)
    assert np.array_equal(got, want)
    # just off the midpoint goes to the nearer neighbour
    assert np.array_equal(xo.double_to_half(np.nextafter(mid, -np.inf)), h)
    assert np.array_equal(xo.double_to_half(np.nextafter(mid, np.inf)), h + 1)
    assert np.array_equal(xo.double_to_half(-mid), want | 0x8000)


def test_fp16_encode_matches_numpy_on_random_doubles():
    rng = np.random.default_rng(3)
    d = np.concatenate([rng.standard_normal(200000) * 10.0 ** rng.integers(-9, 6, 200000),
                        [0.0, -0.0, 65504.0, 65519.9, 65520.0, 1e9, -1e9, 2.0 ** -24, 2.0 ** -25, 2.0 ** -25 * 1.0001,
                         np.inf, -np.inf]])
    with np.errstate(over="ignore"):
        ref = d.astype(np.float16).view(np.uint16)
    assert np.array_equal(xo.double_to_half(d), ref)


# ---------------------------------------------------------------- Table 1

def test_table1_geometry_matches_paper(golden_dir):
    for n, v, wb, used, reserve, _v2, _v2a in read_golden(os.path.join(golden_dir, "table1_packing.txt")):
        n, v, wb, used, reserve = map(int, (n, v, wb, used, reserve))
        assert xo.table1(n) == (v, wb)
        assert v * n == used and wb - used == reserve


def test_table1_v2a_lane_constraint(golden_dir):
    # V2a needs 128 / values_per_word integral and dividing the warp: only N in {2, 4} (Table 1 caption)
    g = {k: float(v) for k, v in read_golden(os.path.join(golden_dir, "storage_arithmetic.txt"))}
    ok = []
    for n, v, *_rest, v2a in read_golden(os.path.join(golden_dir, "table1_packing.txt")):
        n, v = int(n), int(v)
        lanes = 128 / v
        fits = lanes == int(lanes) and 32 % int(lanes) == 0
        assert fits == bool(int(v2a))
        if fits:
            ok.append((n, int(lanes), 32 // int(lanes)))
    assert (4, int(g["lanes_per_group_n4"]), int(g["groups_per_iter_n4"])) in ok
    assert (2, int(g["lanes_per_group_n2"]), int(g["groups_per_iter_n2"])) in ok


def test_table1_hand_worked_words():
    # value j at bits [j*N, (j+1)*N), LSB first, reserve bits zero -- words worked out by hand
    assert xo.table1_pack_row(2, np.arange(16, dtype=np.uint8) % 4)[0] == 0xE4E4E4E4
    assert xo.table1_pack_row(3, np.arange(10, dtype=np.uint8) % 8)[0] == 0x08FAC688
    assert xo.table1_pack_row(3, np.full(10, 7, np.uint8))[0] == 0x3FFFFFFF
    assert xo.table1_pack_row(4, np.arange(1, 9, dtype=np.uint8))[0] == 0x87654321
    assert xo.table1_pack_row(5, np.array([1, 2, 3], np.uint8))[0] == 0x0C41
    assert xo.table1_pack_row(5, np.full(3, 31, np.uint8))[0] == 0x7FFF
    assert xo.table1_pack_row(6, np.arange(1, 6, dtype=np.uint8))[0] == 0x05103081
    assert xo.table1_pack_row(6, np.full(5, 63, np.uint8))[0] == 0x3FFFFFFF


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6])
def test_table1_roundtrip_and_word_counts(bits):
    rng = np.random.default_rng(bits)
    v, wb = xo.table1(bits)
    for cols in (1, v - 1, v, v + 1, 128, 1000, 4096):
        for idx in (rng.integers(0, 1 << bits, cols, dtype=np.uint8), np.full(cols, (1 << bits) - 1, np.uint8)):
            w = xo.table1_pack_row(bits, idx)
            assert w.size == -(-cols // v) and w.dtype.itemsize * 8 == wb
            assert np.array_equal(xo.table1_unpack_row(bits, w, cols), idx)
    # words per row at K = 4096: 256 / 410 / 512 / 1366 / 820
    assert xo.table1_pack_row(bits, np.zeros(4096, np.uint8)).size == {2: 256, 3: 410, 4: 512, 5: 1366, 6: 820}[bits]


def test_storage_arithmetic(golden_dir):
    g = {k: float(v) for k, v in read_golden(os.path.join(golden_dir, "storage_arithmetic.txt"))}
    assert g["outlier_bytes"] == 8 + 8 + 2
    assert abs(g["outlier_bytes"] * g["outlier_cap"] - g["outlier_bytes_per_weight_at_cap"]) < 1e-12
    assert g["v2a_library_bytes_n4"] == 32 * 16 * 2
    # a byte id + fp16 scale + fp16 mid per 128 weights reproduces the printed ~0.31 bit/weight
    assert round((8 + 16 + 16) / 128, 2) == g["v2a_overhead_bits"]
    y = (0.5 + g["outlier_cap"] * g["outlier_bytes"] - 0.375) / g["outlier_bytes"]
    assert round(y, 3) == g["breakeven_outlier_fraction"]


# ---------------------------------------------------------------- dequantisation

def _brute_dense_fp64(q):
    """Independent triple loop over the unpacked tensors -> (real-valued D + S, fp16 W^)."""
    f16 = lambda a: np.asarray(a, np.uint16).view(np.float16)
    D = np.zeros((q.rows, q.cols))
    D16 = np.zeros((q.rows, q.cols), np.float16)
    cb = f16(q.codebook).astype(np.float64)
    for i in range(q.rows):
        for k in range(q.cols):
            j = q.idx[i, k]
            if q.mode == 0:
                D[i, k] = cb[i, j]
                D16[i, k] = f16(q.codebook)[i, j]
            else:
                g = k // q.group_size
                s = f16(q.gscale)[i, g]
                m = f16(q.gmid)[i, g]
                e = f16(q.codebook)[q.gid[i, g], j]
                D[i, k] = float(m) + float(s) * float(e)
                D16[i, k] = np.float16(np.float32(s) * np.float32(e) + np.float32(m))
    S = np.zeros((q.rows, q.cols))
    for i in range(q.rows):
        for p in range(q.rowptr[i], q.rowptr[i + 1]):
            S[i, q.ocol[p]] = float(f16(q.oval)[p])
    W16 = D16.copy()
    nz = S != 0
    W16[nz] = (D16.astype(np.float64)[nz] + S[nz]).astype(np.float16)
    return D + S, W16


@pytest.mark.parametrize("mode,bits", [(0, 2), (0, 3), (0, 4), (0, 5), (0, 6), (1, 2), (1, 3), (1, 4), (1, 6)])
def test_dequant_matches_brute_force(mode, bits):
    q = synth.random_quantized(mode, 12, 256, bits, 0.03, seed=100 + bits + 10 * mode)
    _, W16 = _brute_dense_fp64(q)
    got = xo.dequant(to_oracle(q))
    assert np.array_equal(got, W16.view(np.uint16))


def test_v2a_value_against_exact_rational_arithmetic():
    """scale*lib + mid evaluated exactly, rounded once to fp32 and once to fp16 by integer rules."""
    def rne(fr: Fraction, mant_bits: int, emin: int) -> Fraction:
        if fr == 0:
            return fr
        s, a = (-1 if fr < 0 else 1), abs(fr)
        e = a.numerator.bit_length() - a.denominator.bit_length()
        if Fraction(2) ** e > a:
            e -= 1
        e = max(e, emin)
        ulp = Fraction(2) ** (e - mant_bits)
        n = a / ulp
        fl = n.numerator // n.denominator
        r = n - fl
        if r > Fraction(1, 2) or (r == Fraction(1, 2) and fl % 2 == 1):
            fl += 1
        return s * fl * ulp

    rng = np.random.default_rng(11)
    hs = rng.integers(0, 0x7c00, size=(4000, 3)).astype(np.uint16) | (rng.integers(0, 2, size=(4000, 3)).astype(np.uint16) << 15)
    # include subnormals and tiny values
    hs[:200] &= 0x83ff
    for sc, lb, md in hs:
        f = [Fraction(float(np.uint16(v).view(np.float16))) for v in (sc, lb, md)]
        exact = f[0] * f[1] + f[2]
        r32 = rne(exact, 23, -126)
        r16 = rne(r32, 10, -14)
        want = np.float16(float(r16)) if abs(r16) <= 65504 else np.float16(np.inf if r16 > 0 else -np.inf)
        got = np.uint16(xo.v2a_value16(int(sc), int(lb), int(md))).view(np.float16)
        assert got == want or (got == 0 and want == 0), (sc, lb, md, got, want)


def test_outlier_free_positions_are_bit_copies():
    q = synth.random_quantized(0, 8, 256, 4, 0.02, seed=5)
    got = xo.dequant(to_oracle(q))
    mask = np.zeros((q.rows, q.cols), bool)
    for i in range(q.rows):
        mask[i, q.ocol[q.rowptr[i]:q.rowptr[i + 1]]] = True
    plain = np.take_along_axis(q.codebook, q.idx.astype(np.int64), axis=1)
    assert np.array_equal(got[~mask], plain[~mask])
    assert not np.array_equal(got[mask], plain[mask])


# ---------------------------------------------------------------- fp64 GEMV

@pytest.mark.parametrize("mode,bits", [(0, 3), (0, 4), (0, 5), (1, 2), (1, 4)])
def test_gemv_matches_independent_dense_matvec(mode, bits):
    q = synth.random_quantized(mode, 10, 384, bits, 0.02, seed=40 + bits)
    x16 = synth.activations(3, q.cols, seed=9)
    Wd, _ = _brute_dense_fp64(q)
    x = x16.view(np.float16).astype(np.float64)
    y, a = xo.gemv(to_oracle(q), x16)
    assert np.allclose(y, x @ Wd.T, rtol=1e-12, atol=1e-15)
    assert np.allclose(a, np.abs(x)[:, None, :].__mul__(np.abs(Wd)[None]).sum(-1), rtol=1e-12)


def test_gemv_no_outliers_is_pure_codebook_matvec():
    q = synth.random_quantized(0, 16, 256, 4, 0.0, seed=1)
    assert q.nnz == 0
    x16 = synth.activations(1, q.cols, seed=2)
    cb = q.codebook.view(np.float16).astype(np.float64)
    D = np.take_along_axis(cb, q.idx.astype(np.int64), axis=1)
    y, _ = xo.gemv(to_oracle(q), x16)
    assert np.allclose(y[0], D @ x16.view(np.float16).astype(np.float64)[0], rtol=1e-12)


def test_gemv_single_entry_codebook_is_rank_one():
    # every codebook entry of row i equals c_i  =>  y_i = c_i * sum_k x_k whatever the indices are
    q = synth.random_quantized(0, 16, 512, 4, 0.0, seed=3)
    c = (np.arange(16) - 7.5) * 0.01
    q.codebook = np.repeat(c.astype(np.float16)[:, None], 16, axis=1).copy().view(np.uint16)
    x16 = synth.activations(2, q.cols, seed=4)
    x = x16.view(np.float16).astype(np.float64)
    y, _ = xo.gemv(to_oracle(q), x16)
    want = x.sum(axis=1)[:, None] * c.astype(np.float16).astype(np.float64)[None, :]
    assert np.allclose(y, want, rtol=1e-12, atol=1e-15)


def test_gemv_v2a_constant_library_closed_form():
    # lib == v everywhere  =>  y_i = sum_g (mid_ig + scale_ig * v) * X_g with X_g the group sums of x
    q = synth.random_quantized(1, 8, 512, 4, 0.0, seed=6)
    v = np.float16(0.375)
    q.codebook = np.full_like(q.codebook, v.view(np.uint16))
    x16 = synth.activations(1, q.cols, seed=7)
    x = x16.view(np.float16).astype(np.float64)[0]
    Xg = x.reshape(-1, 128).sum(axis=1)
    w = q.gmid.view(np.float16).astype(np.float64) + q.gscale.view(np.float16).astype(np.float64) * float(v)
    y, _ = xo.gemv(to_oracle(q), x16)
    assert np.allclose(y[0], w @ Xg, rtol=1e-12)


def test_gemv_outlier_only_equals_sparse_matvec():
    for mode in (0, 1):
        q = synth.random_quantized(mode, 32, 256, 4, 0.05, seed=8 + mode)
        if mode == 0:
            q.codebook = np.zeros_like(q.codebook)
        else:
            q.gscale = np.zeros_like(q.gscale)
            q.gmid = np.zeros_like(q.gmid)
        x16 = synth.activations(2, q.cols, seed=10)
        x = x16.view(np.float16).astype(np.float64)
        S = sp.csr_matrix((q.oval.view(np.float16).astype(np.float64), q.ocol, q.rowptr), shape=(q.rows, q.cols))
        y, _ = xo.gemv(to_oracle(q), x16)
        assert np.allclose(y, (S @ x.T).T, rtol=1e-12, atol=1e-15)


def test_gemv_v2a_unit_affine_equals_v2_with_library_rows():
    # scale = 1, mid = 0, every group of row i using entry id_i  ==  V2 whose codebook_i = lib[id_i]
    q = synth.random_quantized(1, 12, 384, 3, 0.01, seed=12)
    ids = (np.arange(q.rows) * 5 % q.lib_size).astype(np.uint8)
    q.gid = np.repeat(ids[:, None], q.cols // 128, axis=1).copy()
    q.gscale = np.full_like(q.gscale, np.float16(1.0).view(np.uint16))
    q.gmid = np.zeros_like(q.gmid)
    v2 = synth.QuantTensors(0, q.rows, q.cols, q.bits, q.idx, q.codebook[ids].copy(), q.rowptr, q.ocol, q.oval)
    x16 = synth.activations(1, q.cols, seed=13)
    ya, aa = xo.gemv(to_oracle(q), x16)
    yb, ab = xo.gemv(to_oracle(v2), x16)
    assert np.array_equal(ya, yb) and np.array_equal(aa, ab)
    assert np.array_equal(xo.dequant(to_oracle(q)), xo.dequant(to_oracle(v2)))


def test_gemv_row_window():
    q = synth.random_quantized(0, 40, 256, 4, 0.01, seed=14)
    x16 = synth.activations(1, q.cols, seed=15)
    full, _ = xo.gemv(to_oracle(q), x16)
    part, _ = xo.gemv(to_oracle(q), x16, 7, 19)
    assert np.array_equal(part[:, 7:19], full[:, 7:19]) and not part[:, :7].any() and not part[:, 19:].any()


def test_gemv_with_real_activations_matches_the_fp16_entry_and_a_dense_matvec():
    """gemv_x64 (activations as doubles, for bf16 inputs) is the same sum as gemv on fp16-representable x,
    and equals a dense numpy matvec on values fp16 cannot hold."""
    from paper_2605_14844_b200 import synth
    from conftest import to_oracle
    for mode in (0, 1):
        q = synth.random_quantized(mode, 48, 384, 4, 0.01, seed=61 + mode)
        m = to_oracle(q)
        x16 = synth.activations(2, 384, seed=62)
        y16, a16 = xo.gemv(m, x16)
        y64, a64 = xo.gemv_x64(m, x16.view(np.float16).astype(np.float64))
        assert np.array_equal(y16, y64) and np.array_equal(a16, a64)
        # bf16-like values outside the fp16 range: 8 significant bits, exponents down to 2^-30 and up to 2^20
        rng = np.random.default_rng(63)
        xr = np.round(rng.uniform(1, 2, (2, 384)) * 128) / 128 * 2.0 ** rng.integers(-30, 21, (2, 384))
        y, a = xo.gemv_x64(m, xr)
        if mode == 0:           # V2: D + S written out densely (the sum before any rounding), then a plain matvec
            cb = q.codebook.view(np.float16).astype(np.float64)
            Wd = np.take_along_axis(cb, q.idx.astype(np.int64), axis=1)
            for i in range(q.rows):
                for p_ in range(q.rowptr[i], q.rowptr[i + 1]):
                    Wd[i, q.ocol[p_]] += float(q.oval[p_:p_ + 1].view(np.float16)[0])
            assert np.allclose(y, (Wd @ xr.T).T, rtol=1e-12, atol=0)
        assert np.all(a >= np.abs(y))


def test_silu_mul_against_closed_forms_and_a_library_sigmoid():
    """The element-wise step of a gated expert block, h = SiLU(gate) * up with SiLU(g) = g * sigmoid(g): exact
    values, both limits, the odd-part identity SiLU(g) - SiLU(-g) = g, a library sigmoid, and the slope bound the
    fused-store tolerance relies on."""
    from scipy.special import expit
    u = np.array([1.0, -2.5, 3.0, 0.125])
    assert np.array_equal(xo.silu_mul(np.zeros(4), u), np.zeros(4))               # SiLU(0) = 0
    assert xo.silu_mul(np.array([1.0]), np.array([1.0]))[0] == pytest.approx(1.0 / (1.0 + np.exp(-1.0)), rel=1e-15)
    assert xo.silu_mul(np.array([np.log(3.0)]), np.array([2.0]))[0] == pytest.approx(2.0 * np.log(3.0) * 0.75, rel=1e-14)
    big = np.array([40.0, 80.0, 700.0])
    assert np.allclose(xo.silu_mul(big, np.ones(3)), big, rtol=1e-15)             # -> g for g >> 0
    assert np.all(np.abs(xo.silu_mul(-big, np.ones(3))) < 1e-15)                  # -> 0 for g << 0
    rng = np.random.default_rng(71)
    g = rng.normal(0, 4, 4096)
    up = rng.normal(0, 2, 4096)
    one = np.ones_like(g)
    assert np.allclose(xo.silu_mul(g, one) - xo.silu_mul(-g, one), g, rtol=0, atol=1e-14)
    assert np.allclose(xo.silu_mul(g, up), expit(g) * g * up, rtol=1e-13, atol=1e-300)
    assert np.allclose(xo.silu_mul(g, 3.0 * up), 3.0 * xo.silu_mul(g, up), rtol=1e-15)   # linear in `up`
    # |SiLU'| <= 1.1 everywhere (the maximum, 1.0998, sits near g = 2.4): central differences on a fine grid
    t = np.linspace(-30, 30, 600001)
    d = (xo.silu_mul(t + 1e-6, np.ones_like(t)) - xo.silu_mul(t - 1e-6, np.ones_like(t))) / 2e-6
    assert 1.099 < np.abs(d).max() <= 1.1 and 2.3 < t[np.argmax(d)] < 2.5
    assert d.min() > -0.1                                                         # the dip left of zero is shallow
