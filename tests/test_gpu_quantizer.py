"""Parity of the GPU encoder (include/xfp_quant.h) against the CPU oracle's encoder, stage by stage.

Stages whose outputs are integers or fp16 values (extraction mask, Lloyd codebooks and indices, LibFit
library / ids / scales / mid-points / indices, residual CSR, median) must match the oracle BIT FOR BIT on
the same inputs: both sides take those decisions in fp64, operation by operation.  The two reductions
whose summation order is the kernel's own (matrix statistics, per-channel cosine) are held to 1e-12
relative; to keep the later stages' inputs identical the tests hand the oracle's (mu, sigma) to both sides.
"""
import ctypes as C
import os

import numpy as np
import pytest
import torch

from oracle import xfp_oracle as xo
import paper_2605_14844_b200 as xfp
from paper_2605_14844_b200 import quant_binding as qb
from paper_2605_14844_b200 import synth

pytestmark = pytest.mark.gpu


def _dev(a):
    a = np.ascontiguousarray(a)
    return torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).cuda()


def _u16(t):
    return t.cpu().numpy().view(np.uint16)


def _ws(rows, cols):
    return torch.empty(qb.xfp_quant_workspace_size(rows, cols) + 256, dtype=torch.uint8, device="cuda")


def _weights(rows, cols, seed, rate=0.01):
    W = synth.gaussian_weights(rows, cols, seed)
    return synth.plant_uniform_outliers(W, rate, seed + 1)


def _ms(mu, sg):
    return torch.tensor([mu, sg], dtype=torch.float64, device="cuda")


# ------------------------------------------------------------------ statistics

@pytest.mark.parametrize("rows,cols", [(96, 512), (1, 128), (333, 1536)])
def test_stats_match_serial_fp64(rows, cols):
    W = _weights(rows, cols, 5)
    mu, sg = xo.stats(W)
    out = torch.zeros(2, dtype=torch.float64, device="cuda")
    qb.xfp_quant_stats(_dev(W), 0, out, _ws(rows, cols))
    got = out.cpu().numpy()
    assert abs(got[0] - mu) <= 1e-12 * max(abs(mu), np.abs(W).mean())
    assert abs(got[1] - sg) <= 1e-12 * sg
    # robust scale: exact selection of the median |w - mu|, so only mu's last bits can differ
    _, _, rs = xo.outlier_mask(W, sigma_mode="robust")
    qb.xfp_quant_stats(_dev(W), 1, out, _ws(rows, cols))
    assert abs(out.cpu().numpy()[1] - rs) <= 1e-10 * rs


# ------------------------------------------------------------------ extraction mask

def _gpu_mask(W, mu, sg, mode, k_or_rate, cap):
    rows, cols = W.shape
    mask = torch.full((rows, cols), 7, dtype=torch.uint8, device="cuda")
    cnt = torch.zeros(2, dtype=torch.int64, device="cuda")
    qb.xfp_quant_outliers(_dev(W), _ms(mu, sg), mode, k_or_rate, cap, mask, cnt, _ws(rows, cols))
    torch.cuda.synchronize()
    return mask.cpu().numpy(), int(cnt[0].item())


@pytest.mark.parametrize("k,cap", [(4.0, 0.02), (4.0, 0.002), (1.0, 0.05), (3.0, 0.0), (50.0, 0.02)])
def test_threshold_mask_is_bit_exact(k, cap):
    W = _weights(160, 640, 11, rate=0.01)
    want, mu, sg = xo.outlier_mask(W, k=k, cap=cap)
    got, cnt = _gpu_mask(W, mu, sg, 0, k, cap)
    assert np.array_equal(got, want)
    assert cnt == int(want.sum())


@pytest.mark.parametrize("rate", [0.0, 0.003, 0.02, 0.5, 1.0])
def test_rate_mask_is_bit_exact(rate):
    W = _weights(96, 1024, 12)
    want, mu, sg = xo.outlier_mask(W, rate=rate)
    got, cnt = _gpu_mask(W, mu, sg, 1, rate, 0.0)
    assert np.array_equal(got, want)
    assert cnt == int(want.sum()) == int(np.floor(rate * W.size))


def test_mask_ties_keep_the_lower_positions():
    # only four distinct |w - mu|: every cut falls inside a run of equal keys
    rng = np.random.default_rng(3)
    W = rng.choice(np.array([-2.0, -1.0, -0.5, 0.5, 1.0, 2.0], dtype=np.float32), size=(64, 512))
    mu, sg = xo.stats(W)
    for rate in (0.1, 0.4, 0.77):
        want, _, _ = xo.outlier_mask(W, rate=rate)
        got, _ = _gpu_mask(W, mu, sg, 1, rate, 0.0)
        assert np.array_equal(got, want)
    want, _, _ = xo.outlier_mask(W, k=0.5, cap=0.3)
    got, cnt = _gpu_mask(W, mu, sg, 0, 0.5, 0.3)
    assert np.array_equal(got, want) and cnt == int(np.floor(0.3 * W.size))


# ------------------------------------------------------------------ Lloyd (V2)

def _gpu_lloyd(W, mask, mu, bits, iters):
    rows, cols = W.shape
    cb = torch.zeros((rows, 1 << bits), dtype=torch.int16, device="cuda")
    idx = torch.full((rows, cols), 255, dtype=torch.uint8, device="cuda")
    qb.xfp_quant_lloyd(_dev(W), None if mask is None else _dev(mask), _ms(mu, 0.0), bits, iters, cb, idx)
    torch.cuda.synchronize()
    return _u16(cb), idx.cpu().numpy()


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6])
@pytest.mark.parametrize("cols,iters", [(512, 20), (1536, 5), (4096, 20)])
def test_lloyd_is_bit_exact(bits, cols, iters):
    rows = 24
    W = _weights(rows, cols, 20 + bits)
    mask, mu, _ = xo.outlier_mask(W)
    m = xo.quantize_v2(W, bits, mask, mu, iters)
    cb, idx = _gpu_lloyd(W, mask, mu, bits, iters)
    assert np.array_equal(cb, m.codebook)
    assert np.array_equal(idx, m.idx)


def test_lloyd_degenerate_channels():
    cols = 256
    rng = np.random.default_rng(8)
    W = np.zeros((6, cols), dtype=np.float32)
    W[0] = 0.125                                              # one value
    W[1] = rng.choice(np.array([-0.5, 0.25, 1.0], dtype=np.float32), cols)   # fewer values than entries
    W[2] = np.linspace(-1, 1, cols, dtype=np.float32)         # uniform
    W[3] = rng.standard_normal(cols).astype(np.float32) * 1e-6
    W[4, ::2] = 3.0                                           # two values, ties at the midpoint entries
    W[5] = rng.standard_normal(cols).astype(np.float32) * 100
    for bits in (2, 4, 6):
        for iters in (0, 1, 20):
            m = xo.quantize_v2(W, bits, np.zeros(W.shape, np.uint8), 0.0, iters)
            cb, idx = _gpu_lloyd(W, None, 0.0, bits, iters)
            assert np.array_equal(cb, m.codebook), (bits, iters)
            assert np.array_equal(idx, m.idx), (bits, iters)


# ------------------------------------------------------------------ LibFit (V2a)

@pytest.mark.parametrize("bits,L,rows", [(2, 32, 96), (3, 32, 200), (4, 32, 64), (4, 7, 40), (3, 32, 20), (6, 16, 48)])
def test_libfit_library_is_bit_exact(bits, L, rows):
    cols = 512
    W = _weights(rows, cols, 40 + bits)
    mask, mu, _ = xo.outlier_mask(W)
    v2 = xo.quantize_v2(W, bits, mask, mu, 20)
    want = np.empty((L, 1 << bits), dtype=np.uint16)
    xo._lib.xo_libfit_library(v2.codebook.reshape(-1), rows, bits, L, 20, want.reshape(-1))
    lib = torch.zeros((L, 1 << bits), dtype=torch.int16, device="cuda")
    qb.xfp_quant_libfit_library(_dev(v2.codebook), rows, bits, L, 20, lib, _ws(rows, cols))
    torch.cuda.synchronize()
    assert np.array_equal(_u16(lib), want)


@pytest.mark.parametrize("bits,group", [(2, 128), (3, 128), (4, 128), (5, 128), (3, 64), (4, 256), (6, 64), (2, 256)])
def test_libfit_assign_is_bit_exact(bits, group):
    """Group assignment at the paper's group size and at the other two the format carries (64, 256)."""
    rows, cols, L = 48, 768, 32
    W = _weights(rows, cols, 50 + bits)
    W[3, 256:512] = 0.0625        # constant groups at every group size
    mask, mu, _ = xo.outlier_mask(W)
    m = xo.quantize_v2a(W, bits, mask, mu, L, 20, group=group)
    G = cols // group
    idx = torch.full((rows, cols), 255, dtype=torch.uint8, device="cuda")
    gid = torch.full((rows, G), 255, dtype=torch.uint8, device="cuda")
    gs = torch.zeros((rows, G), dtype=torch.int16, device="cuda")
    gm = torch.zeros((rows, G), dtype=torch.int16, device="cuda")
    qb.xfp_quant_libfit_assign(_dev(W), _dev(mask), _ms(mu, 0.0), bits, L, _dev(m.codebook), idx, gid, gs, gm,
                               group_size=group)
    torch.cuda.synchronize()
    assert np.array_equal(gid.cpu().numpy(), m.gid)
    assert np.array_equal(_u16(gs), m.gscale)
    assert np.array_equal(_u16(gm), m.gmid)
    assert np.array_equal(idx.cpu().numpy(), m.idx)


# ------------------------------------------------------------------ residual, cosine, median

def _desc(m):
    return xfp.XfpDesc(m.mode, m.rows, m.cols, m.bits, 128, m.lib_size if m.mode else 0, 32, 0)


@pytest.mark.parametrize("mode,bits", [(0, 3), (0, 5), (1, 2), (1, 4)])
def test_residual_and_cosine(mode, bits):
    rows, cols = 80, 768
    W = _weights(rows, cols, 60 + bits, rate=0.02)
    W[7] = 0.0                                   # a zero channel: cosine 1 by definition
    mask, mu, _ = xo.outlier_mask(W, k=3.0)
    mask[11] = 0                                 # a channel with nothing extracted
    m = xo.quantize_v2(W, bits, mask, mu, 5) if mode == 0 else xo.quantize_v2a(W, bits, mask, mu, 32, 5)
    nnz = m.nnz
    Wd, md = _dev(W), _dev(mask)
    args = (_dev(m.idx), _dev(m.codebook), _dev(m.gid) if mode else None, _dev(m.gscale) if mode else None,
            _dev(m.gmid) if mode else None)
    rowptr = torch.zeros(rows + 1, dtype=torch.int32, device="cuda")
    ocol = torch.full((nnz,), -1, dtype=torch.int32, device="cuda")
    oval = torch.zeros(nnz + 8, dtype=torch.int16, device="cuda")[:nnz]
    qb.xfp_quant_residual(_desc(m), Wd, md, *args, rowptr, ocol, oval, _ws(rows, cols))
    torch.cuda.synchronize()
    assert np.array_equal(rowptr.cpu().numpy(), m.rowptr)
    assert np.array_equal(ocol.cpu().numpy(), m.ocol)
    assert np.array_equal(_u16(oval), m.oval)
    # a buffer that is too small drops the tail and still reports the true counts
    small = torch.full((nnz // 2,), -1, dtype=torch.int32, device="cuda")
    sval = torch.zeros(nnz // 2 + 8, dtype=torch.int16, device="cuda")[:nnz // 2]
    qb.xfp_quant_residual(_desc(m), Wd, md, *args, rowptr, small, sval, _ws(rows, cols))
    torch.cuda.synchronize()
    assert int(rowptr[-1].item()) == nnz
    assert np.array_equal(small.cpu().numpy(), m.ocol[:nnz // 2])

    cos = torch.zeros(rows, dtype=torch.float64, device="cuda")
    qb.xfp_quant_cosine(_desc(m), Wd, md, *args, cos)
    want = xo.row_cosine(W, xo.dequant(m))
    got = cos.cpu().numpy()
    assert got[7] == 1.0
    assert np.max(np.abs(got - want)) <= 1e-12
    med = torch.zeros(2, dtype=torch.float64, device="cuda")
    qb.xfp_quant_median(cos, med, _ws(rows, cols))
    assert float(med[0].item()) == xo.median(got)
    odd = cos[:rows - 1].clone()
    qb.xfp_quant_median(odd, med, _ws(rows, cols))
    assert float(med[0].item()) == xo.median(got[:rows - 1])


def test_median_handles_signs_and_duplicates():
    rng = np.random.default_rng(2)
    for n in (1, 2, 5, 1000, 4097, 65536, 65537, 200000):   # one-block kernel up to 65536, device-wide above
        v = np.round(rng.standard_normal(n), 1)          # many duplicates, both signs, zeros
        med = torch.zeros(2, dtype=torch.float64, device="cuda")
        qb.xfp_quant_median(_dev(v), med, _ws(1, 128))
        assert float(med[0].item()) == xo.median(v), n


# ------------------------------------------------------------------ Algorithm 1 end to end

def _params(k=4.0, cap=0.02, rate=None, iters=20, sigma_mode=0):
    return qb.XfpQuantParams(sigma_mode, 0 if rate is None else 1, k, cap, 0.0 if rate is None else rate, iters, 0)


@pytest.mark.parametrize("mode,cands,tau,expect_fallback", [
    (0, (2, 3, 4), 0.96, False), (0, (4, 5), 0.96, False), (0, (2, 3), 0.999, True),
    (1, (2, 4), 0.93, False), (1, (3,), 0.93, False)])
def test_auto_select_matches_the_oracle_and_feeds_the_decode_path(mode, cands, tau, expect_fallback):
    rows, cols, L = 128, 1024, 32
    W = synth.plant_column_outliers(synth.gaussian_weights(rows, cols, 70), 0.01, 71)
    ref = xo.auto_select(W, "attention", cands, tau_strict=tau, mode=mode, iters=20, lib_size=L)
    cap = int(np.floor(0.02 * W.size))
    buf = qb.QuantBuffers(rows, cols, mode, max(cands), L, cap)
    res = qb.xfp_quantize(mode, _dev(W), _params(), cands, tau, buf)
    torch.cuda.synchronize()
    assert res.bits == ref.bits and bool(res.fallback) == ref.info["fallback"] == expect_fallback
    assert res.tried == len(ref.info["tried"])
    assert abs(res.median_cos - ref.info["median_cos"]) <= 1e-12
    assert abs(res.mu - ref.info["mu"]) <= 1e-12 * np.abs(W).mean() and abs(res.sigma - ref.info["sigma"]) <= 1e-12
    E = 1 << res.bits
    nnz = int(res.nnz)
    assert nnz == ref.nnz
    assert np.array_equal(buf.rowptr.cpu().numpy(), ref.rowptr)
    assert np.array_equal(buf.ocol[:nnz].cpu().numpy(), ref.ocol)
    # mu enters Lloyd as the value of the extracted positions; its last bits differ between the serial
    # and the tree sum, which can move a cell mean by one fp64 ulp but, short of an exact fp16 tie, no output
    assert np.array_equal(buf.idx.cpu().numpy(), ref.idx)
    if mode == 0:
        assert np.array_equal(_u16(buf.codebook.view(-1)[:rows * E].view(rows, E)), ref.codebook)
    else:
        assert np.array_equal(_u16(buf.lib.view(-1)[:L * E].view(L, E)), ref.codebook)
        assert np.array_equal(buf.gid.cpu().numpy(), ref.gid)
        assert np.array_equal(_u16(buf.gscale), ref.gscale) and np.array_equal(_u16(buf.gmid), ref.gmid)
    assert np.array_equal(_u16(buf.oval[:nnz]), ref.oval)

    # the tensors go straight into xfp_pack and the fused GEMV, without leaving the device
    desc = xfp.XfpDesc(mode, rows, cols, res.bits, 128, L if mode else 0, 32, nnz)
    pb, wb = xfp.xfp_packed_size(desc)
    packed = torch.empty(pb, dtype=torch.uint8, device="cuda")
    wsp = torch.zeros(max(wb, 16), dtype=torch.uint8, device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    table = buf.lib.view(-1)[:L * E] if mode else buf.codebook.view(-1)[:rows * E]
    xfp.xfp_pack(desc, buf.idx, table.contiguous(), buf.gid, buf.gscale, buf.gmid, buf.rowptr, buf.ocol, buf.oval,
                 packed, err)
    x16 = synth.activations(1, cols, 72)
    xd = torch.from_numpy(np.ascontiguousarray(x16).view(np.int16)).cuda().view(torch.float16).reshape(1, cols)
    y = torch.empty((1, rows), dtype=torch.float32, device="cuda")
    (xfp.xfp_gemv_v2a if mode else xfp.xfp_gemv_v2)(desc, packed, xd, 1, y, False, wsp)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    yref, absum = xo.gemv(ref, np.ascontiguousarray(x16).view(np.uint16).reshape(1, cols))
    assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - yref) <= 1e-3 * absum + 1e-30)


@pytest.mark.parametrize("mode,cands,tau", [(1, (2, 3, 4), 0.95), (1, (2, 4), 0.93), (0, (2, 3, 4), 0.95)])
def test_moe_sampling_layer_matches_the_oracle(mode, cands, tau):
    """MoE sampling ("Auto-Selection"): Algorithm 1 on four stacked experts, then every expert of the layer encoded at
    that width (V2a: against the sample's library).  Same width, same median, same library bits as the oracle, and
    every expert's packed blob reconstructs to the oracle's matrix bit for bit and decodes inside the GEMV bound."""
    rows, cols, L = 64, 512, 32
    experts = [synth.plant_uniform_outliers(synth.gaussian_weights(rows, cols, 800 + e) * np.float32(1.0 + 0.07 * e),
                                            0.004, 900 + e) for e in range(6)]
    sample = (1, 2, 4, 5)
    ref, info = xo.auto_select_moe(experts, sample, candidates=cands, tau=tau, mode=mode, lib_size=L)
    pms, res, lib = qb.quantize_moe_layer([_dev(W) for W in experts], mode, cands, tau, sample, _params(), L)
    torch.cuda.synchronize()
    assert res.bits == info["bits"] and bool(res.fallback) == info["fallback"]
    assert abs(res.median_cos - info["median_cos"]) <= 1e-12
    if mode:
        assert np.array_equal(_u16(lib), ref[0].codebook)
    x16 = synth.activations(2, cols, 77)
    xd = torch.from_numpy(np.ascontiguousarray(x16).view(np.int16)).cuda().view(torch.float16)
    for pm, q in zip(pms, ref):
        assert pm.desc.bits == q.bits and int(pm.desc.nnz) == q.nnz and int(pm.err_word.item()) == 0
        assert np.array_equal(_u16(pm.dequant().view(torch.int16)), xo.dequant(q))
        yref, absum = xo.gemv(q, np.ascontiguousarray(x16).view(np.uint16))
        y = pm.gemv(xd)
        torch.cuda.synchronize()
        assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - yref) <= 1e-3 * absum + 1e-30)


@pytest.mark.parametrize("group,cands", [(64, (2, 4)), (256, (3,))])
def test_auto_select_at_other_group_sizes(group, cands):
    """Algorithm 1 for V2a with 64 and 256 weights per group: same width and tensors as the oracle, and the packed blob
    reconstructs to the oracle's matrix bit for bit."""
    rows, cols, L = 96, 1024, 32
    W = synth.plant_uniform_outliers(synth.gaussian_weights(rows, cols, 75), 0.005, 76)
    ref = xo.auto_select(W, "moe_routed", cands, tau_lazy=0.93, mode=1, iters=20, lib_size=L, group=group)
    params = _params()
    params.group_size = group
    pm, res = qb.quantize_and_pack(_dev(W), 1, cands, 0.93, params, lib_size=L)
    torch.cuda.synchronize()
    assert res.bits == ref.bits and int(res.nnz) == ref.nnz and abs(res.median_cos - ref.info["median_cos"]) <= 1e-12
    assert pm.desc.group_size == group and int(pm.err_word.item()) == 0
    assert np.array_equal(_u16(pm.dequant().view(torch.int16)), xo.dequant(ref))


def test_quantize_reports_a_small_outlier_buffer():
    rows, cols = 64, 512
    W = _weights(rows, cols, 90, rate=0.02)
    buf = qb.QuantBuffers(rows, cols, 0, 4, 0, 16)
    with pytest.raises(xfp.XfpError):
        qb.xfp_quantize(0, _dev(W), _params(), (4,), 0.9, buf)


# ------------------------------------------------------------------ the paper's layer sizes

@pytest.mark.parametrize("mode,rows,cols,bits", [(0, 4096, 4096, 4), (1, 3072, 4096, 3)])
def test_full_size_layers_are_bit_exact(mode, rows, cols, bits):
    """A dense-attention projection (V2, heavy outlier columns) and a routed expert's gate_up projection (V2a)
    at the sizes the decode benchmarks use, every output of every stage compared in full."""
    L = 32
    if mode == 0:
        W = synth.attention_weights(10, rows, cols)
    else:
        W = synth.plant_uniform_outliers(synth.gaussian_weights(rows, cols, 30), 0.001, 31)
    mask, mu, sg = xo.outlier_mask(W)
    ref = xo.quantize_v2(W, bits, mask, mu, 20) if mode == 0 else xo.quantize_v2a(W, bits, mask, mu, L, 20)
    Wd, msd, ws = _dev(W), _ms(mu, sg), _ws(rows, cols)
    maskd = torch.empty((rows, cols), dtype=torch.uint8, device="cuda")
    cnt = torch.zeros(2, dtype=torch.int64, device="cuda")
    qb.xfp_quant_outliers(Wd, msd, 0, 4.0, 0.02, maskd, cnt, ws)
    assert np.array_equal(maskd.cpu().numpy(), mask)
    E = 1 << bits
    cb = torch.empty((rows, E), dtype=torch.int16, device="cuda")
    idx = torch.empty((rows, cols), dtype=torch.uint8, device="cuda")
    qb.xfp_quant_lloyd(Wd, maskd, msd, bits, 20, cb, idx)
    gid = gs = gm = None
    table = cb
    if mode:
        G = cols // 128
        lib = torch.empty((L, E), dtype=torch.int16, device="cuda")
        gid = torch.empty((rows, G), dtype=torch.uint8, device="cuda")
        gs = torch.empty((rows, G), dtype=torch.int16, device="cuda")
        gm = torch.empty((rows, G), dtype=torch.int16, device="cuda")
        qb.xfp_quant_libfit_library(cb, rows, bits, L, 20, lib, ws)
        qb.xfp_quant_libfit_assign(Wd, maskd, msd, bits, L, lib, idx, gid, gs, gm)
        table = lib
        assert np.array_equal(gid.cpu().numpy(), ref.gid)
        assert np.array_equal(_u16(gs), ref.gscale) and np.array_equal(_u16(gm), ref.gmid)
    assert np.array_equal(_u16(table), ref.codebook)
    assert np.array_equal(idx.cpu().numpy(), ref.idx)
    nnz = ref.nnz
    rowptr = torch.empty(rows + 1, dtype=torch.int32, device="cuda")
    ocol = torch.empty(nnz, dtype=torch.int32, device="cuda")
    oval = torch.empty(nnz + 8, dtype=torch.int16, device="cuda")[:nnz]
    desc = xfp.XfpDesc(mode, rows, cols, bits, 128, L if mode else 0, 32, 0)
    qb.xfp_quant_residual(desc, Wd, maskd, idx, table, gid, gs, gm, rowptr, ocol, oval, ws)
    assert np.array_equal(rowptr.cpu().numpy(), ref.rowptr)
    assert np.array_equal(ocol.cpu().numpy(), ref.ocol) and np.array_equal(_u16(oval), ref.oval)
    cos = torch.empty(rows, dtype=torch.float64, device="cuda")
    qb.xfp_quant_cosine(desc, Wd, maskd, idx, table, gid, gs, gm, cos)
    assert np.max(np.abs(cos.cpu().numpy() - xo.row_cosine(W, xo.dequant(ref)))) <= 1e-12


@pytest.mark.parametrize("mode", [0, 1])
def test_float_weights_to_decode_in_one_call(mode):
    """quantize_and_pack: float weights -> packed blob on the device; y = W^ x must then be close to W x in the way
    the cosine gate promises, and xfp_dequant of the blob must equal the oracle's reconstruction of the same matrix."""
    rows, cols = 256, 1024
    W = synth.plant_column_outliers(synth.gaussian_weights(rows, cols, 95), 0.01, 96)
    pm, res = qb.quantize_and_pack(_dev(W), mode, (3, 4), 0.96)
    ref = xo.auto_select(W, "attention", (3, 4), tau_strict=0.96, mode=mode, iters=20, lib_size=32)
    assert res.bits == ref.bits and int(pm.err_word.item()) == 0
    got = pm.dequant()
    torch.cuda.synchronize()
    assert np.array_equal(_u16(got), xo.dequant(ref))
    x16 = synth.activations(1, cols, seed=97)
    y = pm.gemv(torch.from_numpy(x16.view(np.int16)).cuda().view(torch.float16)).cpu().numpy().astype(np.float64)[0]
    exact = W.astype(np.float64) @ x16.view(np.float16).astype(np.float64)[0]
    cos = float(y @ exact / (np.linalg.norm(y) * np.linalg.norm(exact)))
    assert cos > 0.99


@pytest.mark.parametrize("cols,bits,iters", [(28672, 4, 20), (16512, 3, 5), (65536, 5, 5)])
def test_lloyd_on_channels_too_long_for_shared_memory(cols, bits, iters):
    """Above 16384 weights per channel the sorted arrays live in global scratch; the results are the same bits."""
    rows = 10
    W = _weights(rows, cols, 120 + bits)
    mask, mu, _ = xo.outlier_mask(W)
    m = xo.quantize_v2(W, bits, mask, mu, iters)
    cb = torch.zeros((rows, 1 << bits), dtype=torch.int16, device="cuda")
    idx = torch.full((rows, cols), 255, dtype=torch.uint8, device="cuda")
    qb.xfp_quant_lloyd(_dev(W), _dev(mask), _ms(mu, 0.0), bits, iters, cb, idx, _ws(rows, cols))
    torch.cuda.synchronize()
    assert np.array_equal(_u16(cb), m.codebook)
    assert np.array_equal(idx.cpu().numpy(), m.idx)
    with pytest.raises(xfp.XfpError):          # the workspace is not optional here
        qb.xfp_quant_lloyd(_dev(W), _dev(mask), _ms(mu, 0.0), bits, iters, cb, idx, None)


def test_auto_select_on_a_wide_matrix():
    rows, cols = 320, 28672        # more channels than resident CTAs: every CTA walks several
    W = synth.plant_column_outliers(synth.gaussian_weights(rows, cols, 130), 0.005, 131)
    ref = xo.auto_select(W, "attention", (4,), tau_strict=0.9, iters=5)
    pm, res = qb.quantize_and_pack(_dev(W), 0, (4,), 0.9, qb.XfpQuantParams(0, 0, 4.0, 0.02, 0.0, 5, 0))
    got = pm.dequant()
    torch.cuda.synchronize()
    assert int(res.nnz) == ref.nnz and np.array_equal(_u16(got), xo.dequant(ref))


def _random_encoder_cases(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(count):
        out.append((i, int(rng.integers(0, 2)), int(rng.choice([1, 5, 33, 64, 130, 300])), 128 * int(rng.choice([1, 2, 3, 7, 12, 20])),
                    tuple(sorted(set(int(b) for b in rng.integers(2, 7, size=int(rng.integers(1, 4)))))),
                    float(rng.choice([0.5, 0.93, 0.96, 0.99, 0.9999])), int(rng.choice([0, 1, 5, 20])),
                    int(rng.integers(0, 2)), int(rng.integers(0, 2)), int(rng.choice([1, 5, 32, 40]))))
    return out


@pytest.mark.parametrize("case", _random_encoder_cases(int(os.environ.get("XFP_SWEEP_CASES", "72")) // 2, 777 + int(os.environ.get("XFP_SWEEP_SEED", "0"))),
                         ids=lambda c: "-".join(str(v) for v in c))
def test_randomized_auto_select(case):
    """A seeded sweep of Algorithm 1 end to end against the oracle: mode, ragged channel counts, channel lengths,
    candidate lists, floors that pass early, late or never, 0..20 Lloyd rounds, both sigma modes, both extraction
    modes, library sizes including ones larger than the channel count."""
    i, mode, rows, cols, cands, tau, iters, sigma_mode, outlier_mode, L = case
    W = synth.plant_uniform_outliers(synth.gaussian_weights(rows, cols, 8000 + i), 0.01, 8100 + i)
    rate = 0.004 if outlier_mode else None
    ref = xo.auto_select(W, "attention", cands, tau_strict=tau, mode=mode, k=3.0, cap=0.01,
                         sigma_mode="robust" if sigma_mode else "matrix", rate=rate, iters=iters, lib_size=L)
    params = qb.XfpQuantParams(sigma_mode, outlier_mode, 3.0, 0.01, 0.004, iters, 0)
    buf = qb.QuantBuffers(rows, cols, mode, max(cands), L, int(0.02 * W.size) + 8)
    res = qb.xfp_quantize(mode, _dev(W), params, cands, tau, buf)
    torch.cuda.synchronize()
    assert (res.bits, bool(res.fallback), res.tried) == (ref.bits, ref.info["fallback"], len(ref.info["tried"]))
    E, nnz = 1 << res.bits, int(res.nnz)
    assert nnz == ref.nnz and np.array_equal(buf.mask.cpu().numpy(), _oracle_mask(W, ref))
    assert np.array_equal(buf.idx.cpu().numpy(), ref.idx)
    table = buf.lib.view(-1)[:L * E].view(L, E) if mode else buf.codebook.view(-1)[:rows * E].view(rows, E)
    assert np.array_equal(_u16(table), ref.codebook)
    if mode:
        assert np.array_equal(buf.gid.cpu().numpy(), ref.gid)
        assert np.array_equal(_u16(buf.gscale), ref.gscale) and np.array_equal(_u16(buf.gmid), ref.gmid)
    assert np.array_equal(buf.rowptr.cpu().numpy(), ref.rowptr)
    assert np.array_equal(buf.ocol[:nnz].cpu().numpy(), ref.ocol) and np.array_equal(_u16(buf.oval[:nnz]), ref.oval)
    assert abs(res.median_cos - ref.info["median_cos"]) <= 1e-12


def _oracle_mask(W, ref):
    m = np.zeros(W.shape, dtype=np.uint8)
    for r in range(ref.rows):
        m[r, ref.ocol[ref.rowptr[r]:ref.rowptr[r + 1]]] = 1
    return m
