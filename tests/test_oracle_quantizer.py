"""Pins for the oracle's encoder half: outlier extraction, per-channel Lloyd, the cosine gate
and auto-select (Algorithm 1), LibFit.

The Lloyd pins are closed forms (uniform source), textbook Lloyd-Max distortions (Gaussian
source, tests/golden/lloyd_max_gaussian.txt), exact recovery of discrete sources, and the
paper's printed XFP3 bulk cosines.  LibFit: the group assignment is checked against exhaustive search and
the library against k-means fixed-point invariants; the paper prints no V2a figure, so the reading of LibFit
itself stays unpinned against the paper.
"""
import os

import numpy as np
import pytest

from conftest import read_golden
from oracle import xfp_oracle as xo
from paper_2605_14844_b200 import synth


def _f16(a):
    return np.asarray(a, np.uint16).view(np.float16).astype(np.float64)


# ---------------------------------------------------------------- outlier extraction

def test_outlier_mask_equals_brute_force_predicate():
    W = synth.config1_weights(seed=21, rows=64, cols=512)
    mask, mu, sg = xo.outlier_mask(W, k=4.0, cap=0.02)
    Wd = W.astype(np.float64)
    assert abs(mu - Wd.mean()) < 1e-15 and abs(sg - Wd.std()) < 1e-14   # population std
    assert np.array_equal(mask.astype(bool), np.abs(Wd - mu) > 4.0 * sg)
    assert 0 < mask.mean() <= 0.02


def test_outlier_cap_keeps_largest_with_index_tiebreak():
    rng = np.random.default_rng(5)
    W = rng.standard_normal((32, 256)).astype(np.float32)
    W[3, 10] = W[1, 7] = 9.0           # an exact tie in |w - mu| is impossible to guarantee after the mean
    mask, mu, sg = xo.outlier_mask(W, k=1.0, cap=0.02)     # k=1 would take ~32 %; the cap bites
    keep = int(np.floor(0.02 * W.size))
    assert mask.sum() == keep
    key = np.abs(W.astype(np.float64) - mu).reshape(-1)
    order = np.lexsort((np.arange(key.size), -key))        # by key descending, then flat index ascending
    assert np.array_equal(np.flatnonzero(mask.reshape(-1)), np.sort(order[:keep]))


def test_outlier_top_rate_is_exact():
    W = synth.gaussian_weights(48, 512, seed=9)
    for rate in (0.0, 0.003, 0.02):
        mask, mu, _ = xo.outlier_mask(W, rate=rate)
        keep = int(np.floor(rate * W.size))
        assert mask.sum() == keep
        if keep:
            key = np.abs(W.astype(np.float64) - mu)
            assert key[mask.astype(bool)].min() >= key[~mask.astype(bool)].max()


def test_robust_sigma_sees_the_bulk():
    W = synth.config1_weights(seed=2, rows=256, cols=1024)
    _, _, sg_matrix = xo.outlier_mask(W)
    mask, _, sg_robust = xo.outlier_mask(W, k=6.0, sigma_mode="robust")
    assert abs(sg_robust - 0.02) < 0.0005 < sg_matrix - 0.02          # the planted tail inflates the plain sigma
    assert abs(mask.mean() - 0.003) < 2e-4                            # k=6 on the bulk sigma takes the planted set


def test_residual_reconstructs_outliers_to_half_an_ulp():
    W = synth.config1_weights(seed=4, rows=64, cols=512)
    mask, mu, _ = xo.outlier_mask(W, k=4.0)
    m = xo.quantize_v2(W, 4, mask, mu)
    assert m.nnz == mask.sum()
    rec = _f16(xo.dequant(m))
    pos = mask.astype(bool)
    w = W.astype(np.float64)[pos]
    # two fp16 roundings (the residual, then the sum): within one fp16 ulp of the original
    ulp = np.spacing(np.abs(w).astype(np.float16)).astype(np.float64)
    assert np.all(np.abs(rec[pos] - w) <= ulp)
    # CSR is well formed: ascending columns in every row, positions = the mask
    for i in range(m.rows):
        c = m.ocol[m.rowptr[i]:m.rowptr[i + 1]]
        assert np.all(np.diff(c) > 0) and np.array_equal(c, np.flatnonzero(mask[i]))


# ---------------------------------------------------------------- Lloyd

@pytest.mark.parametrize("bits", [2, 3, 4])
def test_lloyd_uniform_source_closed_form(bits):
    # uniform on [-1, 1]: the optimal quantiser is the uniform one, D = (2/2^N)^2 / 12, and
    # cos = sqrt(1 - D/var) with var = 1/3  =>  sqrt(1 - 2^-2N)
    K = 1 << 16
    v = (np.arange(K) + 0.5) / K * 2.0 - 1.0
    cb, idx, _, trace = xo.lloyd_row(v, bits, iters=50, want_trace=True)
    rec = _f16(cb)[idx]
    cos = rec @ v / np.linalg.norm(rec) / np.linalg.norm(v)
    assert abs(cos - np.sqrt(1 - 2.0 ** (-2 * bits))) < 2e-4
    step = 2.0 / (1 << bits)
    assert np.allclose(_f16(cb), -1 + step * (np.arange(1 << bits) + 0.5), atol=2e-3)
    assert abs(trace[-1] - step * step / 12) < 1e-5


def test_lloyd_gaussian_source_reaches_lloyd_max(golden_dir):
    rng = np.random.default_rng(17)
    v = rng.standard_normal(400000)
    for n, levels, dist in read_golden(os.path.join(golden_dir, "lloyd_max_gaussian.txt")):
        n, dist = int(n), float(dist)
        cb, idx, _, trace = xo.lloyd_row(v, n, iters=400, want_trace=True)
        assert abs(trace[-1] / v.var() - dist) < 0.03 * dist + 2e-4, (n, trace[-1])


def test_lloyd_distortion_never_increases_and_entries_are_cell_means():
    rng = np.random.default_rng(23)
    v = rng.standard_normal(4096) * 0.02
    cb, idx, done, trace = xo.lloyd_row(v, 4, iters=20, want_trace=True)
    assert np.all(np.diff(trace) <= 1e-18)
    c = _f16(cb)
    assert np.all(np.diff(c) >= 0)
    # every stored index is the nearest stored entry (ties to the lower index)
    d = np.abs(v[:, None] - c[None, :])
    assert np.array_equal(idx, d.argmin(axis=1))
    # run to convergence: each entry equals the mean of the values assigned to it (up to the fp16
    # rounding of the entries, which also moves a few values across cell borders)
    cb, idx, done, _ = xo.lloyd_row(v, 3, iters=500, want_trace=True)
    assert done < 500
    c = _f16(cb)
    for j in range(8):
        sel = v[idx == j]
        assert sel.size and abs(sel.mean() - c[j]) <= 2e-5        # values have sigma 0.02


def test_lloyd_discrete_source_is_exact():
    rng = np.random.default_rng(29)
    levels = np.array([-0.75, -0.25, 0.125, 0.5])                     # fp16-exact values
    v = levels[rng.integers(0, 4, 4096)]
    for bits in (2, 3):
        cb, idx, _ = xo.lloyd_row(v, bits, iters=20)
        assert np.array_equal(_f16(cb)[idx], v)


def test_lloyd_first_round_uses_cdf_quantile_init():
    # with zero rounds the codebook is the initialisation: entry j = sorted[floor((j+0.5) K / 2^N)]
    rng = np.random.default_rng(31)
    v = rng.standard_normal(1000)
    cb, _, done = xo.lloyd_row(v, 3, iters=0)
    s = np.sort(v)
    want = s[np.floor((np.arange(8) + 0.5) * 1000 / 8).astype(int)].astype(np.float16)
    assert done == 0 and np.array_equal(cb.view(np.float16), want)


def test_gaussian_rows_reproduce_paper_xfp3_bulk_cosine(golden_dir):
    """On near-Gaussian layers the paper prints XFP3 bulk cosines of 0.980-0.983; per-channel Lloyd
    with quantile initialisation on Gaussian rows must land in the same band (5 to 20 rounds)."""
    printed = [float(r[2]) for r in read_golden(os.path.join(golden_dir, "paper_bulk_cosine.txt"))]
    W = synth.gaussian_weights(256, 4096, seed=33)
    none = np.zeros(W.shape, np.uint8)
    for iters, want in ((5, 0.9808), (20, 0.9825)):
        m = xo.quantize_v2(W, 3, none, 0.0, iters=iters)
        med = xo.median(xo.row_cosine(W, xo.dequant(m)))
        assert abs(med - want) < 0.001
        assert min(printed) - 0.001 <= med <= max(printed) + 0.001


@pytest.mark.parametrize("bits,want", [(2, 0.9393), (4, 0.9946), (5, 0.9980)])
def test_gaussian_rows_cosine_at_twenty_rounds(bits, want):
    # sqrt(1 - D) for the textbook distortions is the ceiling; 20 rounds from the quantile start sit just under
    W = synth.gaussian_weights(128, 4096, seed=35)
    m = xo.quantize_v2(W, bits, np.zeros(W.shape, np.uint8), 0.0, iters=20)
    med = xo.median(xo.row_cosine(W, xo.dequant(m)))
    ceiling = {2: np.sqrt(1 - 0.1175), 4: np.sqrt(1 - 0.009497), 5: np.sqrt(1 - 0.002499)}[bits]
    assert abs(med - want) < 0.001 and med <= ceiling + 5e-4


# ---------------------------------------------------------------- cosine gate and auto-select

def test_row_cosine_and_median():
    rng = np.random.default_rng(37)
    W = rng.standard_normal((5, 64)).astype(np.float32)
    R = (W * np.float32(1.5)).astype(np.float16)
    R[1] = -R[1]
    W[4] = 0
    cosv = xo.row_cosine(W, R.view(np.uint16))
    Rd = R.astype(np.float64)
    for i in range(4):
        want = W[i].astype(np.float64) @ Rd[i] / np.linalg.norm(W[i].astype(np.float64)) / np.linalg.norm(Rd[i])
        assert abs(cosv[i] - want) < 1e-12
    assert cosv[1] < -0.99 and cosv[4] == 1.0
    assert xo.median(np.array([3.0, 1.0, 2.0])) == 2.0 and xo.median(np.array([4.0, 1.0, 2.0, 3.0])) == 2.5


def test_auto_select_on_gaussian_rows_brackets_the_paper():
    W = synth.gaussian_weights(64, 4096, seed=41)
    picks = {}
    for tau in (0.93, 0.95, 0.96, 0.98, 0.99):
        m = xo.auto_select(W, "attention", candidates=(2, 3, 4), tau_strict=tau, k=4.0)
        picks[tau] = m.bits
        assert not m.info["fallback"] and m.info["median_cos"] >= tau
        # the next smaller candidate (if any) failed the floor
        for n, med in m.info["tried"][:-1]:
            assert med < tau
    assert picks == {0.93: 2, 0.95: 3, 0.96: 3, 0.98: 3, 0.99: 4}
    # the lazy floor applies to routed experts only; the strict one to everything else
    lazy = xo.auto_select(W, "moe_routed", candidates=(2, 4), tau_strict=0.96, tau_lazy=0.93, mode=xo.MODE_V2)
    strict = xo.auto_select(W, "shared_expert", candidates=(2, 4), tau_strict=0.96, tau_lazy=0.93, mode=xo.MODE_V2)
    assert (lazy.bits, strict.bits) == (2, 4) and lazy.info["tau"] == 0.93 and strict.info["tau"] == 0.96


def test_auto_select_falls_back_to_largest_candidate():
    W = synth.gaussian_weights(32, 1024, seed=43)
    m = xo.auto_select(W, candidates=(2, 3), tau_strict=0.999)
    assert m.bits == 3 and m.info["fallback"] and m.info["median_cos"] < 0.999


def test_outlier_extraction_raises_cosine_on_heavy_tailed_layer():
    # the effect Table 4 reports for attention layers: bulk-only reconstruction is worse than bulk + outliers
    W = synth.attention_weights(seed=45, rows=128, cols=2048)
    mask, mu, _ = xo.outlier_mask(W, k=4.0)
    none = np.zeros_like(mask)
    with_out = xo.median(xo.row_cosine(W, xo.dequant(xo.quantize_v2(W, 3, mask, mu))))
    without = xo.median(xo.row_cosine(W, xo.dequant(xo.quantize_v2(W, 3, none, mu))))
    assert with_out > without + 0.005


# ---------------------------------------------------------------- LibFit (no figure in the paper to pin the reading)

def test_libfit_sanity():
    W = synth.gaussian_weights(96, 1024, seed=47)
    mask, mu, _ = xo.outlier_mask(W, rate=0.001)
    v2 = xo.quantize_v2(W, 4, mask, mu)
    va = xo.quantize_v2a(W, 4, mask, mu, lib_size=32)
    assert va.codebook.shape == (32, 16) and va.gid.max() < 32 and va.idx.max() < 16
    lib = _f16(va.codebook)
    assert np.all(np.diff(lib, axis=1) >= 0) and np.abs(lib).max() <= 1.0 + 1e-3
    assert np.all(_f16(va.gscale) >= 0)
    Wd = W.astype(np.float64)
    sse2 = ((_f16(xo.dequant(v2)) - Wd) ** 2).sum()
    ssea = ((_f16(xo.dequant(va)) - Wd) ** 2).sum()
    cos2 = xo.median(xo.row_cosine(W, xo.dequant(v2)))
    cosa = xo.median(xo.row_cosine(W, xo.dequant(va)))
    assert cosa > 0.985 and abs(cosa - cos2) < 0.006
    # a constant group decodes exactly
    Wc = W.copy()
    Wc[5, 128:256] = np.float32(0.03125)
    vc = xo.quantize_v2a(Wc, 2, np.zeros(W.shape, np.uint8), 0.0, lib_size=8)
    assert vc.gscale[5, 1] == 0 and np.all(_f16(xo.dequant(vc))[5, 128:256] == 0.03125)
    assert sse2 > 0 and ssea > 0


def _decoded(scale16, lib16, mid16):
    """fp16(fp32(scale*lib + mid)) with numpy's own conversions: the fp16 x fp16 product is exact in fp32."""
    s = np.asarray(scale16, np.uint16).view(np.float16).astype(np.float32)
    l = np.asarray(lib16, np.uint16).view(np.float16).astype(np.float32)
    m = np.asarray(mid16, np.uint16).view(np.float16).astype(np.float32)
    return (s * l + m).astype(np.float16).astype(np.float64)


def _check_assignment_by_exhaustive_search(m, bulk, group):
    """Every group of `m` against exhaustive search over the library `m.codebook`: the stored (mid, scale) are the
    fp16 roundings of the range's middle and half-width, no other library entry gives a smaller squared error
    under nearest-value decoding (ties: the lower entry), and every index points at a nearest decoded value
    (ties: the lower index)."""
    L = m.codebook.shape[0]
    ar = np.arange(group)
    for i in range(m.rows):
        for g in range(m.cols // group):
            v = bulk[i, g * group:(g + 1) * group]
            lo, hi = v.min(), v.max()
            assert m.gmid[i, g] == np.float16(0.5 * (hi + lo)).view(np.uint16)
            assert m.gscale[i, g] == np.float16(0.5 * (hi - lo)).view(np.uint16)
            sse = np.empty(L)
            for l in range(L):
                dec = _decoded(m.gscale[i, g], m.codebook[l], m.gmid[i, g])
                sse[l] = (np.abs(v[:, None] - dec[None, :]).min(axis=1) ** 2).sum()
            chosen = int(m.gid[i, g])
            assert sse[chosen] <= sse.min() * (1 + 1e-12)
            assert chosen == int(np.flatnonzero(sse <= sse.min() * (1 + 1e-12))[0])
            dec = _decoded(m.gscale[i, g], m.codebook[chosen], m.gmid[i, g])
            dist = np.abs(v[:, None] - dec[None, :])
            q = m.idx[i, g * group:(g + 1) * group].astype(int)
            assert np.array_equal(dist[ar, q], dist.min(axis=1))
            assert np.array_equal(q, dist.argmin(axis=1))


@pytest.mark.parametrize("bits,L", [(2, 8), (3, 32), (4, 16)])
def test_libfit_assignment_is_the_brute_force_optimum(bits, L):
    """Second half of LibFit against exhaustive search (group size 128, the paper's default)."""
    rows, cols = 12, 512
    W = synth.plant_uniform_outliers(synth.gaussian_weights(rows, cols, seed=81), 0.01, 82)
    mask, mu, _ = xo.outlier_mask(W)
    m = xo.quantize_v2a(W, bits, mask, mu, lib_size=L)
    _check_assignment_by_exhaustive_search(m, np.where(mask != 0, mu, W.astype(np.float64)), 128)


@pytest.mark.parametrize("group", [64, 256])
def test_libfit_assignment_at_other_group_sizes(group):
    """The group size is a parameter of the format ("Lane geometry"): the same exhaustive-search property at 64
    and 256 weights per group, and the metadata has one (id, scale, mid) per group of that size."""
    rows, cols, bits, L = 10, 1024, 3, 16
    W = synth.plant_uniform_outliers(synth.gaussian_weights(rows, cols, seed=91), 0.01, 92)
    mask, mu, _ = xo.outlier_mask(W)
    m = xo.quantize_v2a(W, bits, mask, mu, lib_size=L, group=group)
    assert m.group_size == group and m.gid.shape == (rows, cols // group)
    _check_assignment_by_exhaustive_search(m, np.where(mask != 0, mu, W.astype(np.float64)), group)
    # the reconstruction uses the group of the stored size: dequant against the decode written out here
    D = _f16(xo.dequant(xo.QuantizedMatrix(m.mode, m.rows, m.cols, m.bits, m.idx, m.codebook,
                                           np.zeros(rows + 1, np.int32), np.zeros(0, np.int32),
                                           np.zeros(0, np.uint16), group_size=group, lib_size=L, gid=m.gid,
                                           gscale=m.gscale, gmid=m.gmid)))
    for i in (0, rows - 1):
        for g in (0, cols // group - 1):
            dec = _decoded(m.gscale[i, g], m.codebook[m.gid[i, g]], m.gmid[i, g])
            assert np.array_equal(D[i, g * group:(g + 1) * group], dec[m.idx[i, g * group:(g + 1) * group]])


def test_libfit_with_a_library_learned_on_another_matrix():
    """The experts of a routed layer share one library ("V2a: Shared Codebook Library"): a library learned on
    matrix A and handed to the quantiser of matrix B is stored unchanged, and B's group assignment against it
    satisfies the same exhaustive-search property as an own library."""
    bits, L = 3, 16
    A = synth.gaussian_weights(48, 512, seed=85)
    B = synth.plant_uniform_outliers(synth.gaussian_weights(12, 512, seed=86) * np.float32(1.7), 0.01, 87)
    ma = xo.quantize_v2a(A, bits, np.zeros(A.shape, np.uint8), 0.0, lib_size=L)
    mask, mu, _ = xo.outlier_mask(B)
    mb = xo.quantize_v2a(B, bits, mask, mu, library=ma.codebook)
    assert mb.lib_size == L and np.array_equal(mb.codebook, ma.codebook)
    assert mb.gid.max() < L and mb.idx.max() < (1 << bits)
    _check_assignment_by_exhaustive_search(mb, np.where(mask != 0, mu, B.astype(np.float64)), 128)
    # a borrowed library must still reconstruct a Gaussian bulk to the 3-bit band
    cos_shared = xo.median(xo.row_cosine(B, xo.dequant(mb)))
    assert cos_shared > 0.975


@pytest.mark.parametrize("mode", [xo.MODE_V2, xo.MODE_V2A])
def test_moe_sampling_selects_on_a_few_experts_and_quantises_all(mode):
    """MoE sampling ("Auto-Selection"): the width comes from Algorithm 1 on the stacked sample alone -- experts outside
    the sample cannot change it -- and every expert, sampled or not, is then quantised on its own at that width:
    the sample's decision reproduces as a plain auto_select on the stacked matrix, a V2 expert equals its stand-alone
    quantisation, and a V2a expert keeps the sample's library unchanged and satisfies the exhaustive-search property
    of the group assignment against it.  Near-Gaussian experts need 3 bits for the 0.93 floor of routed layers
    (2 bits reach 0.9394 only when converged; the sample's median decides), and widening the outsiders by 3x leaves
    the choice alone."""
    rows, cols, L = 24, 512, 16
    experts = [synth.gaussian_weights(rows, cols, seed=700 + e) * np.float32(1.0 + 0.1 * e) for e in range(6)]
    sample = (0, 2, 3, 5)
    qs, info = xo.auto_select_moe(experts, sample, candidates=(2, 3, 4), tau=0.95, mode=mode, lib_size=L)
    stacked = np.concatenate([experts[i] for i in sample], axis=0)
    alone = xo.auto_select(stacked, "moe_routed", (2, 3, 4), tau_lazy=0.95, mode=mode, lib_size=L)
    assert info["bits"] == alone.bits == 3 and not info["fallback"]
    assert info["median_cos"] == alone.info["median_cos"] and info["sample"] == sample
    assert len(qs) == len(experts)
    for W, q in zip(experts, qs):
        mask, mu, _ = xo.outlier_mask(W)
        assert q.bits == 3 and q.rows == rows and q.nnz == int(mask.sum())
        if mode == xo.MODE_V2:
            own = xo.quantize_v2(W, 3, mask, mu)
            assert np.array_equal(q.idx, own.idx) and np.array_equal(q.codebook, own.codebook)
        else:
            assert np.array_equal(q.codebook, alone.codebook)      # the layer's one library
            _check_assignment_by_exhaustive_search(q, np.where(mask != 0, mu, W.astype(np.float64)), 128)
        assert xo.median(xo.row_cosine(W, xo.dequant(q))) > 0.97
    outsiders = [W if e in sample else W * np.float32(3.0) for e, W in enumerate(experts)]
    _, info2 = xo.auto_select_moe(outsiders, sample, candidates=(2, 3, 4), tau=0.95, mode=mode, lib_size=L)
    assert info2["bits"] == info["bits"] and info2["median_cos"] == info["median_cos"]


def test_libfit_library_invariants():
    """First half of LibFit (k-means over normalised codebooks) by what any correct run must satisfy: every
    normalised codebook spans [-1, 1] exactly at its ends, so every centroid does; entries ascend; after
    enough rounds each centroid is the mean of the codebooks nearest to it (a k-means fixed point); and the
    library beats its own starting point."""
    rows, bits, L = 160, 3, 8
    W = synth.gaussian_weights(rows, 1024, seed=83)
    W *= np.linspace(0.5, 2.0, rows, dtype=np.float32)[:, None]          # channels of different scale
    v2 = xo.quantize_v2(W, bits, np.zeros(W.shape, np.uint8), 0.0, 20)
    E = 1 << bits
    lib16 = np.empty((L, E), dtype=np.uint16)
    xo._lib.xo_libfit_library(v2.codebook.reshape(-1), rows, bits, L, 200, lib16.reshape(-1))
    lib = _f16(lib16)
    assert np.all(lib[:, 0] == -1.0) and np.all(lib[:, -1] == 1.0)
    assert np.all(np.diff(lib, axis=1) >= 0)
    c = _f16(v2.codebook)
    mid, half = 0.5 * (c.max(1) + c.min(1)), 0.5 * (c.max(1) - c.min(1))
    u = (c - mid[:, None]) / half[:, None]
    d = ((u[:, None, :] - lib[None, :, :]) ** 2).sum(-1)
    near = d.argmin(1)
    for l in range(L):
        members = u[near == l]
        if len(members):
            assert np.max(np.abs(members.mean(0) - lib[l])) <= 2e-3       # fp16 rounding of entries in [-1, 1]
    one = np.empty((L, E), dtype=np.uint16)
    xo._lib.xo_libfit_library(v2.codebook.reshape(-1), rows, bits, L, 0, one.reshape(-1))   # the seeding alone
    d0 = ((u[:, None, :] - _f16(one)[None, :, :]) ** 2).sum(-1).min(1).sum()
    assert d.min(1).sum() < d0
