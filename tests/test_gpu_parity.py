"""Parity of the CUDA path against the CPU oracle, through the C ABI.

xfp_dequant must match the oracle bit for bit.  The fused GEMV must satisfy
    max_i |y_i - y_ref_i| <= 1e-3 * sum_k |W_ik x_k|
(the tolerance the benchmark spec states; fp32 accumulation of exact products sits far inside it).
"""
import os

import numpy as np
import pytest
import torch

from conftest import from_oracle, to_oracle
from oracle import xfp_oracle as xo
import paper_2605_14844_b200 as xfp
from paper_2605_14844_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-3


def _x_dev(x16):
    return torch.from_numpy(x16.view(np.int16)).cuda().view(torch.float16)


def _check_gemv(q, pm, x16, y_fp16=False, rows=None):
    """Run the GEMV and compare against the oracle (all rows, or the sampled `rows`)."""
    xd = _x_dev(x16)
    y = pm.gemv(xd, y_fp16=y_fp16)
    torch.cuda.synchronize()
    got = y.float().cpu().numpy().astype(np.float64)
    m = to_oracle(q)
    if rows is None:
        ref, absum = xo.gemv(m, x16)
        sel = slice(None)
    else:
        ref = np.zeros((x16.shape[0], q.rows)); absum = np.zeros_like(ref)
        for r in rows:
            yr, ar = xo.gemv(m, x16, int(r), int(r) + 1)
            ref[:, r] = yr[:, r]; absum[:, r] = ar[:, r]
        sel = np.asarray(rows)
    err = np.abs(got[:, sel] - ref[:, sel])
    bound = TOL * absum[:, sel]
    assert np.all(np.isfinite(got[:, sel]))
    assert np.all(err <= bound + 1e-30), float((err / (bound + 1e-30)).max())
    return float((err / (bound + 1e-300)).max()), y


def _check_dequant(q, pm):
    W = pm.dequant()
    torch.cuda.synchronize()
    got = W.view(torch.int16).cpu().numpy().view(np.uint16)
    want = xo.dequant(to_oracle(q))
    assert np.array_equal(got, want)
    assert int(pm.err_word.item()) == 0


CASES = [(mode, bits) for mode in (0, 1) for bits in (2, 3, 4, 5, 6)]


@pytest.mark.parametrize("mode,bits", CASES)
def test_dequant_bit_exact_small(mode, bits):
    # 70 rows: three row-blocks with a ragged tail; 384 columns: three super-chunks
    q = synth.random_quantized(mode, 70, 384, bits, 0.02, seed=500 + 10 * mode + bits)
    _check_dequant(q, xfp.pack_tensors(q))


@pytest.mark.parametrize("mode,bits", CASES)
@pytest.mark.parametrize("batch", [1, 3, 16])
def test_gemv_within_bound_small(mode, bits, batch):
    q = synth.random_quantized(mode, 70, 640, bits, 0.02, seed=600 + 10 * mode + bits)
    pm = xfp.pack_tensors(q, col_bits=16 if bits % 2 else 32)
    x16 = synth.activations(batch, q.cols, seed=77 + batch)
    _check_gemv(q, pm, x16)
    _check_gemv(q, pm, x16, y_fp16=True)


@pytest.mark.parametrize("mode,bits,rows,cols", [(0, 4, 2048, 4096), (1, 3, 2048, 1536), (1, 4, 640, 8192), (0, 6, 96, 12288)])
def test_one_workspace_serves_every_kernel_in_turn(mode, bits, rows, cols):
    """The header's promise: one workspace serves any batch and every GEMV entry point of a shape, one call after the
    other.  Every kernel must leave the counter region zero-filled and must not keep data where another kernel
    keeps counters: a call sequence over ONE workspace (batch 1, 16, 2, 5, bf16, batch 1 again) gives bit for bit what
    the same calls give with a fresh workspace each."""
    q = synth.random_quantized(mode, rows, cols, bits, 0.004, seed=8500 + bits)
    pm = xfp.pack_tensors(q, col_bits=16)
    shared = pm.workspace
    seq = [(1, torch.float16), (16, torch.float16), (2, torch.float16), (5, torch.float16), (3, torch.bfloat16),
           (1, torch.float16), (13, torch.float16), (1, torch.float16)]
    for i, (batch, xdt) in enumerate(seq):
        x = _x_dev(synth.activations(batch, cols, seed=8600 + i)).to(xdt)
        y_shared = torch.empty((batch, rows), dtype=torch.float32, device="cuda")
        y_fresh = torch.empty((batch, rows), dtype=torch.float32, device="cuda")
        xfp.xfp_gemv_typed(pm.desc, pm.packed, x, batch, y_shared, shared)
        xfp.xfp_gemv_typed(pm.desc, pm.packed, x, batch, y_fresh, torch.zeros_like(shared))
        torch.cuda.synchronize()
        assert torch.equal(y_shared, y_fresh), (i, batch)
    counters = shared[:((rows + 31) // 32) * 4].view(torch.int32)
    assert int((counters != 0).sum()) == 0


@pytest.mark.parametrize("group", [64, 256])
@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6])
def test_v2a_group_sizes_other_than_128(group, bits):
    """The group size is a parameter of the format ("Lane geometry"): V2a blobs with 64 and 256 weights per
    (id, scale, mid).  Reconstruction is bit-exact and the fused GEMV stays inside the bound at batch 1, 2, 5 and
    16 -- groups of 256 on the fast kernels (their metadata is stored with both super-chunks), groups of 64 on the
    general one -- and the prefill form agrees too."""
    rows, cols = 200, 1024
    q = synth.random_quantized(1, rows, cols, bits, 0.01, seed=8100 + 10 * bits + group, group_size=group)
    assert q.gid.shape == (rows, cols // group)
    pm = xfp.pack_tensors(q, col_bits=16)
    assert pm.desc.group_size == group
    _check_dequant(q, pm)
    for batch in (1, 2, 5, 16):
        _check_gemv(q, pm, synth.activations(batch, cols, seed=8200 + batch))
    if bits <= 5:
        x40 = synth.activations(40, cols, seed=8300)
        ws = torch.zeros(xfp.xfp_gemm_workspace_size(pm.desc, 40), dtype=torch.uint8, device="cuda")
        y = torch.empty((40, rows), dtype=torch.float32, device="cuda")
        xfp.xfp_gemm(pm.desc, pm.packed, _x_dev(x40), y, ws)
        torch.cuda.synchronize()
        assert int(ws[:4].view(torch.int32).item()) == 0
        ref, absum = xo.gemv(to_oracle(q), x40)
        assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - ref) <= TOL * absum + 1e-30)


def test_group_size_of_a_v2_blob_only_constrains_the_columns():
    q = synth.random_quantized(0, 64, 512, 4, 0.01, seed=8400, group_size=256)
    pm = xfp.pack_tensors(q)
    _check_dequant(q, pm)
    _check_gemv(q, pm, synth.activations(1, 512, seed=8401))


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("rows,cols", [(1, 128), (33, 128), (256, 1536), (96, 12288), (2048, 4096)])
def test_gemv_shapes_and_split_k(mode, rows, cols):
    q = synth.random_quantized(mode, rows, cols, 4, 0.01, seed=rows + cols + mode)
    pm = xfp.pack_tensors(q)
    for batch in (1, 2):
        _check_gemv(q, pm, synth.activations(batch, cols, seed=5))
    _check_dequant(q, pm)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("rows,cols,bits", [(33, 128, 4), (256, 1536, 3), (2048, 4096, 4), (640, 2048, 5)])
def test_batched_shapes_and_split_k(mode, rows, cols, bits):
    """Batches 5 and 12 (a partial tile; a full tile plus a partial one) on shapes whose blocks are cut along K."""
    q = synth.random_quantized(mode, rows, cols, bits, 0.01, seed=3 * rows + cols + mode)
    pm = xfp.pack_tensors(q, col_bits=16)
    for batch in (5, 12):
        _check_gemv(q, pm, synth.activations(batch, cols, seed=50 + batch))
        _check_gemv(q, pm, synth.activations(batch, cols, seed=60 + batch), y_fp16=True)
    tickets = pm.workspace[: ((q.rows + 31) // 32) * 4].view(torch.int32)
    assert int(tickets.abs().sum().item()) == 0


@pytest.mark.parametrize("mode,bits,group", [(0, 2, 128), (0, 3, 128), (0, 4, 128), (0, 5, 128), (0, 6, 128),
                                             (1, 2, 128), (1, 3, 128), (1, 4, 128), (1, 5, 128), (1, 6, 128),
                                             (1, 4, 64), (1, 2, 256), (1, 6, 64)])
def test_several_rows_of_x_on_matrices_of_one_round(mode, bits, group):
    """2..16 rows of x on a matrix of 79 row-blocks (more than half the SMs, fewer than all: one resident CTA per
    row-block, the last one ragged), the shape class on which the one-channel-per-lane kernel with 2, 4 or 8 B
    fragments per decoded fragment takes most batches (all of them at N = 6, up to 4 rows otherwise; the kernels with
    two channels per lane take the rest): tiles of 2, 4 and 8 rows, partial tiles (3, 7), two launches (11, 16)."""
    rows, cols = 2500, 768
    q = synth.random_quantized(mode, rows, cols, bits, 0.015, seed=9100 + 10 * bits + mode + group, group_size=group)
    pm = xfp.pack_tensors(q, col_bits=16)
    for batch in (2, 3, 4, 7, 8, 11, 16):
        _check_gemv(q, pm, synth.activations(batch, cols, seed=9200 + batch), y_fp16=bool(batch & 1))
    tickets = pm.workspace[: ((rows + 31) // 32) * 4].view(torch.int32)
    assert int(tickets.abs().sum().item()) == 0


@pytest.mark.parametrize("mode,bits,rows,cols", [(0, 6, 9600, 2048), (0, 5, 9700, 1024), (1, 4, 19200, 512), (1, 2, 9600, 2048),
                                                 (1, 6, 4800, 1024), (1, 3, 19000, 512)])
def test_several_rows_of_x_with_resident_ctas_and_a_cut_tail(mode, bits, rows, cols):
    """More row-blocks than CTA slots: resident CTAs walk several row-blocks with one staged copy of x, and the blocks
    of the last partial round are cut along K and meet in the workspace (300 or 600 row-blocks on 148 or 296 slots).
    Repeating the call gives the same bits; the counters are left zero."""
    q = synth.random_quantized(mode, rows, cols, bits, 0.01, seed=9300 + bits + rows, placement="clustered")
    pm = xfp.pack_tensors(q, col_bits=16)
    sample = _sample_rows(rows, 96, seed=9301)
    for batch in (2, 4, 5, 8, 12):
        x16 = synth.activations(batch, cols, seed=9400 + batch)
        _, y0 = _check_gemv(q, pm, x16, rows=sample)
        y1 = pm.gemv(_x_dev(x16))
        torch.cuda.synchronize()
        assert torch.equal(y0, y1)
    tickets = pm.workspace[: ((rows + 31) // 32) * 4].view(torch.int32)
    assert int(tickets.abs().sum().item()) == 0


@pytest.mark.parametrize("bits,lib_size", [(2, 1), (2, 7), (2, 33), (2, 64), (3, 5), (4, 1), (4, 33), (4, 64), (4, 200),
                                           (5, 31), (6, 7), (6, 33), (6, 64)])
def test_v2a_library_sizes(bits, lib_size):
    """Library sizes other than the paper's 32: odd counts (the last table word holds one id), a single entry, sizes
    whose tables outgrow shared memory and fall to other kernels; batch 1 and 4, two shapes (a matrix of one round of
    CTAs and one of several), reconstruction bit-exact."""
    for rows, cols in ((2500, 512), (9600, 256)):
        q = synth.random_quantized(1, rows, cols, bits, 0.01, seed=9900 + 10 * bits + lib_size, lib_size=lib_size)
        pm = xfp.pack_tensors(q, col_bits=16)
        sample = _sample_rows(rows, 64, seed=9901)
        for batch in (1, 4):
            _check_gemv(q, pm, synth.activations(batch, cols, seed=9910 + batch), rows=sample)
    _check_dequant(q, pm)


@pytest.mark.parametrize("mode,bits", [(0, 4), (0, 5), (1, 3), (1, 4)])
def test_longest_rows(mode, bits):
    """K = 65536, the largest the descriptor admits (u16 outlier columns): x alone is 128 KB per batch row."""
    q = synth.random_quantized(mode, 40, 65536, bits, 0.005, seed=77 + bits + mode)
    pm = xfp.pack_tensors(q, col_bits=16)
    for batch in (1, 2, 3):
        _check_gemv(q, pm, synth.activations(batch, q.cols, seed=70 + batch))
    _check_dequant(q, pm)


@pytest.mark.parametrize("placement,rate", [("uniform", 0.0), ("clustered", 0.02), ("one_row", 0.01)])
def test_outlier_structures(placement, rate):
    for mode in (0, 1):
        q = synth.random_quantized(mode, 128, 1024, 4, rate, seed=31 + mode, placement=placement)
        pm = xfp.pack_tensors(q, col_bits=16)
        _check_gemv(q, pm, synth.activations(2, q.cols, seed=6))
        _check_dequant(q, pm)


def test_adversarial_activations():
    q = synth.random_quantized(0, 64, 1024, 4, 0.01, seed=91)
    qa = synth.random_quantized(1, 64, 1024, 3, 0.01, seed=92)
    K = q.cols
    f16 = lambda a: np.ascontiguousarray(np.asarray(a, np.float32).astype(np.float16)).view(np.uint16).reshape(1, K)
    hot = np.zeros(K); hot[517] = 3.0
    alt = np.where(np.arange(K) % 2 == 0, 1.0, -1.0)
    tiny = np.full(K, 6e-8)            # fp16 subnormals
    big = np.full(K, 60000.0)          # near the fp16 maximum
    for x in (np.ones(K), alt, hot, tiny, big, np.zeros(K)):
        for qq in (q, qa):
            _check_gemv(qq, xfp.pack_tensors(qq), f16(x))


def test_gemv_is_deterministic_and_leaves_workspace_clean():
    q = synth.random_quantized(0, 256, 4096, 4, 0.01, seed=93)
    pm = xfp.pack_tensors(q)
    xd = _x_dev(synth.activations(1, q.cols, seed=8))
    y1 = pm.gemv(xd).clone()
    y2 = pm.gemv(xd).clone()
    torch.cuda.synchronize()
    assert torch.equal(y1, y2)
    tickets = pm.workspace[: ((q.rows + 31) // 32) * 4].view(torch.int32)
    assert int(tickets.abs().sum().item()) == 0


def test_encoder_output_round_trip():
    """Weights -> oracle encoder (outliers, Lloyd, auto-select) -> xfp_pack -> GPU; both modes."""
    W = synth.config1_weights(seed=1, rows=192, cols=1024)
    m = xo.auto_select(W, "attention", candidates=(3, 4), tau_strict=0.96, k=6.0, sigma_mode="robust")
    q = from_oracle(m)
    pm = xfp.pack_tensors(q)
    _check_dequant(q, pm)
    _check_gemv(q, pm, synth.activations(1, q.cols, seed=2))
    mask, mu, _ = xo.outlier_mask(W, rate=0.001)
    ma = xo.quantize_v2a(W, 3, mask, mu, lib_size=32)
    qa = from_oracle(ma)
    pa = xfp.pack_tensors(qa)
    _check_dequant(qa, pa)
    _check_gemv(qa, pa, synth.activations(1, qa.cols, seed=3))


def test_pack_reports_bad_data_and_stays_safe():
    q = synth.random_quantized(1, 64, 256, 3, 0.02, seed=95)
    bad = synth.QuantTensors(**{**q.__dict__})
    bad.idx = q.idx.copy(); bad.idx[3, 7] = 9                # >= 2^3
    bad.gid = q.gid.copy(); bad.gid[5, 1] = 200              # >= L
    bad.ocol = q.ocol.copy()
    if q.rowptr[1] - q.rowptr[0] >= 2:
        bad.ocol[q.rowptr[0] + 1] = bad.ocol[q.rowptr[0]]    # not strictly ascending
    bad.ocol[-1] = 70000                                      # >= cols
    pm = xfp.pack_tensors(bad)
    torch.cuda.synchronize()
    err = int(pm.err_word.item())
    assert err & 1 and err & 2 and err & 8
    y = pm.gemv(_x_dev(synth.activations(1, q.cols, seed=4)))   # must run without faulting
    torch.cuda.synchronize()
    assert torch.isfinite(y).all()


def test_grouped_matches_single_calls():
    n, rows, cols = 8, 160, 1536
    qs = [synth.random_quantized(1, rows, cols, 3, 0.001, seed=700 + j) for j in range(n)]
    for q in qs[1:]:
        q.codebook = qs[0].codebook               # one library per layer, shared by its experts
    pms = [xfp.pack_tensors(q, col_bits=16) for q in qs]
    xs = [_x_dev(synth.activations(1, cols, seed=800 + j)) for j in range(n)]
    ys = torch.zeros((n, rows), dtype=torch.float32, device="cuda")
    d0 = pms[0].desc
    # one descriptor for the group: same shape and mode; nnz = the largest count of the group
    desc = xfp.XfpDesc(d0.mode, d0.rows, d0.cols, d0.bits, d0.group_size, d0.lib_size, d0.col_bits,
                       max(p.desc.nnz for p in pms))
    _, wb = xfp.xfp_packed_size(desc)
    ws = torch.zeros(n * wb, dtype=torch.uint8, device="cuda")
    ptr = lambda ts: torch.tensor([t.data_ptr() for t in ts], dtype=torch.int64, device="cuda")
    xfp.xfp_gemv_grouped(desc, n, ptr([p.packed for p in pms]), ptr(xs), ptr([ys[j] for j in range(n)]), False, ws)
    torch.cuda.synchronize()
    for j in range(n):
        single = pms[j].gemv(xs[j])
        ref, absum = xo.gemv(to_oracle(qs[j]), xs[j].view(torch.int16).cpu().numpy().view(np.uint16))
        # the single call may split K differently from the group launch: both obey the bound, and they
        # agree with each other far inside it
        assert np.all(np.abs(ys[j].cpu().numpy() - ref[0]) <= TOL * absum[0])
        assert np.all(np.abs(single[0].cpu().numpy() - ref[0]) <= TOL * absum[0])
        assert np.all(np.abs(single[0].cpu().numpy() - ys[j].cpu().numpy()) <= 0.05 * TOL * absum[0])


@pytest.mark.parametrize("mode,bits", [(0, 4), (0, 6), (1, 5), (1, 6)])
def test_grouped_other_modes(mode, bits):
    """Grouped launches outside the routed-MoE mode: V2 blobs (every blob its own codebooks) and wide V2a."""
    n, rows, cols = 5, 224, 640
    qs = [synth.random_quantized(mode, rows, cols, bits, 0.004 * (j + 1), seed=1500 + 11 * j + bits) for j in range(n)]
    if mode == 1:
        for q in qs[1:]:
            q.codebook = qs[0].codebook
    pms = [xfp.pack_tensors(q, col_bits=32) for q in qs]
    x16s = [synth.activations(1, cols, seed=1600 + j) for j in range(n)]
    xs = [_x_dev(x) for x in x16s]
    ys = torch.full((n, rows), float("nan"), dtype=torch.float16, device="cuda")
    d0 = pms[0].desc
    desc = xfp.XfpDesc(d0.mode, d0.rows, d0.cols, d0.bits, d0.group_size, d0.lib_size, d0.col_bits,
                       max(p.desc.nnz for p in pms))
    _, wb = xfp.xfp_packed_size(desc)
    ws = torch.zeros(n * wb, dtype=torch.uint8, device="cuda")
    ptr = lambda ts: torch.tensor([t.data_ptr() for t in ts], dtype=torch.int64, device="cuda")
    xfp.xfp_gemv_grouped(desc, n, ptr([p.packed for p in pms]), ptr(xs), ptr([ys[j] for j in range(n)]), True, ws)
    torch.cuda.synchronize()
    for j in range(n):
        ref, absum = xo.gemv(to_oracle(qs[j]), x16s[j])
        assert np.all(np.abs(ys[j].float().cpu().numpy().astype(np.float64) - ref[0]) <= TOL * absum[0])


@pytest.mark.parametrize("bits", [2, 3])
def test_grouped_v2a_many_items_and_mixed_libraries(bits):
    """More work items than resident CTAs (every CTA walks several blocks of several blobs), and blobs
    whose libraries differ: the tables must follow the blob."""
    n, rows, cols = 6, 2112, 384            # 33 blocks of 64 channels per blob, 198 items in all
    qs = [synth.random_quantized(1, rows, cols, bits, 0.002, seed=1300 + j) for j in range(n)]
    qs[1].codebook = qs[0].codebook          # blobs 0, 1 share a library, 2 and 3 share another, 4 and 5 their own
    qs[3].codebook = qs[2].codebook
    pms = [xfp.pack_tensors(q, col_bits=16) for q in qs]
    x16s = [synth.activations(1, cols, seed=1400 + (j // 3)) for j in range(n)]   # two distinct x
    xs = [_x_dev(x) for x in x16s]
    xs = [xs[0], xs[0], xs[0], xs[3], xs[3], xs[3]]
    ys = torch.full((n, rows), float("nan"), dtype=torch.float32, device="cuda")
    d0 = pms[0].desc
    desc = xfp.XfpDesc(d0.mode, d0.rows, d0.cols, d0.bits, d0.group_size, d0.lib_size, d0.col_bits,
                       max(p.desc.nnz for p in pms))
    _, wb = xfp.xfp_packed_size(desc)
    ws = torch.zeros(n * wb, dtype=torch.uint8, device="cuda")
    ptr = lambda ts: torch.tensor([t.data_ptr() for t in ts], dtype=torch.int64, device="cuda")
    for _ in range(2):
        xfp.xfp_gemv_grouped(desc, n, ptr([p.packed for p in pms]), ptr(xs), ptr([ys[j] for j in range(n)]), False, ws)
    torch.cuda.synchronize()
    for j in range(n):
        ref, absum = xo.gemv(to_oracle(qs[j]), x16s[0 if j < 3 else 3])
        assert np.all(np.abs(ys[j].cpu().numpy() - ref[0]) <= TOL * absum[0])


@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("mode,batch", [(0, 2), (1, 1), (0, 5)])
def test_gemv_host_entry(pinned, mode, batch):
    """Host buffers: pinned (used in place by the device) and pageable (copied)."""
    q = synth.random_quantized(mode, 96, 512, 5 if mode == 0 else 3, 0.01, seed=97)
    pm = xfp.pack_tensors(q)
    x16 = synth.activations(batch, q.cols, seed=9)
    xh = torch.from_numpy(x16.view(np.int16).copy())
    yh = torch.full((batch, q.rows), float("nan"), dtype=torch.float32)
    if pinned:
        xh, yh = xh.pin_memory(), yh.pin_memory()
    xd = torch.empty((batch, q.cols), dtype=torch.int16, device="cuda")
    yd = torch.empty((batch, q.rows), dtype=torch.float32, device="cuda")
    for _ in range(2):
        xfp.xfp_gemv_host(pm.desc, pm.packed, xh, xd, batch, yh, yd, False, pm.workspace)
    torch.cuda.synchronize()
    ref, absum = xo.gemv(to_oracle(q), x16)
    assert np.all(np.abs(yh.numpy() - ref) <= TOL * absum)


# ---------------------------------------------------------------- full-size configurations

def _sample_rows(rows, n, seed):
    rng = np.random.default_rng(seed)
    return np.unique(np.concatenate([[0, 31, 32, rows - 1], rng.integers(0, rows, n)]))


def test_config1_full_size_encoder_to_gpu():
    """4096 x 4096, V2 N=4, 0.3 % planted outliers, robust 6-sigma extraction: the whole chain."""
    W = synth.config1_weights(seed=1)
    mask, mu, _ = xo.outlier_mask(W, k=6.0, sigma_mode="robust")
    m = xo.quantize_v2(W, 4, mask, mu)
    q = from_oracle(m)
    pm = xfp.pack_tensors(q, col_bits=16)
    _check_dequant(q, pm)
    x16 = synth.activations(1, 4096, seed=2)
    worst, y = _check_gemv(q, pm, x16)
    y16 = pm.gemv(_x_dev(x16), y_fp16=True)
    torch.cuda.synchronize()
    assert torch.equal(y16, y.half())
    assert worst < 0.05           # fp32 accumulation sits far inside the 1e-3 bound


@pytest.mark.parametrize("mode,rows,cols,bits,rate", [
    (0, 4096, 4096, 5, 0.01),      # attention block member at 5 bits
    (1, 3072, 4096, 3, 0.001),     # MoE gate_up expert
    (1, 4096, 1536, 3, 0.001),     # MoE down expert
    (0, 8192, 8192, 4, 0.003),     # sweep shape
    (0, 12288, 4096, 6, 0.02),     # decoder MLP up, widest codebook, highest outlier rate
    (1, 4096, 12288, 2, 0.005),    # decoder MLP down, K = 12288
])
def test_full_size_sampled_rows(mode, rows, cols, bits, rate):
    q = synth.random_quantized(mode, rows, cols, bits, rate, seed=rows + bits)
    pm = xfp.pack_tensors(q, col_bits=16)
    sample = _sample_rows(rows, 200, seed=bits)
    _check_gemv(q, pm, synth.activations(1, cols, seed=3), rows=sample)
    # dequant: the sampled rows, bit for bit
    W = pm.dequant()
    torch.cuda.synchronize()
    got = W[torch.from_numpy(sample).cuda()].view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got, xo.dequant(to_oracle(q))[sample])


@pytest.mark.parametrize("mode,batch,rate,placement", [(0, 1, 0.02, "clustered"), (0, 16, 0.003, "uniform"),
                                                        (1, 2, 0.003, "uniform"), (1, 8, 0.02, "clustered")])
def test_sweep_shape_28672x8192_sampled_rows(mode, batch, rate, placement):
    """The large shape of the batch sweep in the launch configurations the timing runs use: 4-bit, V2 and V2a,
    whole rounds of CTAs plus the tiers of K slices; sampled rows against the oracle for every batch row."""
    rows, cols = 28672, 8192
    q = synth.random_quantized(mode, rows, cols, 4, rate, seed=4242 + mode, placement=placement)
    pm = xfp.pack_tensors(q, col_bits=16)
    sample = _sample_rows(rows, 96, seed=batch)
    sample = np.unique(np.concatenate([sample, [18943, 18944, 28640, 28671]]))   # around the cut blocks and the end
    _check_gemv(q, pm, synth.activations(batch, cols, seed=30 + batch), rows=sample)
    tickets = pm.workspace[: ((rows + 31) // 32) * 4].view(torch.int32)
    assert int(tickets.abs().sum().item()) == 0



def _group_desc(pms):
    d0 = pms[0].desc
    return xfp.XfpDesc(d0.mode, d0.rows, d0.cols, d0.bits, d0.group_size, d0.lib_size, d0.col_bits,
                       max(p.desc.nnz for p in pms))


@pytest.mark.parametrize("bits,n,rows_gu,hidden", [(3, 8, 256, 512), (2, 3, 2304, 384), (4, 4, 256, 256), (5, 2, 768, 128),
                                                 (3, 8, 3072, 4096)])
@pytest.mark.parametrize("y_fp16", [True, False])
def test_fused_expert_block(bits, n, rows_gu, hidden, y_fp16):
    """A routed expert block in two launches: gate_up with SiLU(gate)*up in its store, down with the
    routing-weighted sum over the experts in its store.

    Stage 1 is compared with the oracle's fp64 h = SiLU(g)*u under the bound propagated through the
    activation: |SiLU'| <= 1.1, so |dh| <= 1.1 |u| e_g + |SiLU(g)| e_u + one output rounding, with e = 1e-3 sum|W x|
    of the gate and up channel.  Stage 2 takes the GPU's own h as its input on both sides and must obey
    1e-3 * sum_j |w_j| sum_k |W_jik h_jk|."""
    inter = rows_gu // 2
    gus = [synth.random_quantized(1, rows_gu, hidden, bits, 0.002, seed=2100 + j) for j in range(n)]
    dns = [synth.random_quantized(1, hidden, inter, bits, 0.002, seed=2200 + j) for j in range(n)]
    for q in gus[1:]:
        q.codebook = gus[0].codebook
    for q in dns[1:]:
        q.codebook = dns[0].codebook
    pg = [xfp.pack_tensors(q, col_bits=16) for q in gus]
    pd = [xfp.pack_tensors(q, col_bits=16) for q in dns]
    x16 = synth.activations(1, hidden, seed=2300)
    xd = _x_dev(x16)
    ptr = lambda ts: torch.tensor([t.data_ptr() for t in ts], dtype=torch.int64, device="cuda")
    dt = torch.float16 if y_fp16 else torch.float32
    h = torch.full((n, inter), float("nan"), dtype=dt, device="cuda")
    dg, dd = _group_desc(pg), _group_desc(pd)
    wsg = torch.zeros(n * xfp.xfp_packed_size(dg)[1], dtype=torch.uint8, device="cuda")
    wsd = torch.zeros(n * xfp.xfp_packed_size(dd)[1], dtype=torch.uint8, device="cuda")
    for _ in range(2):      # twice: the counters must come back to zero
        xfp.xfp_gemv_grouped_epilogue(dg, n, ptr([p.packed for p in pg]), ptr([xd] * n), ptr([h[j] for j in range(n)]),
                                      y_fp16, xfp.XFP_EPI_SWIGLU, None, wsg)
    torch.cuda.synchronize()
    hg = h.float().cpu().numpy().astype(np.float64)
    blocks = rows_gu // 64
    gate_rows = (np.arange(blocks)[:, None] * 64 + np.arange(32)[None, :]).reshape(-1)
    for j in range(n):
        ref, absum = xo.gemv(to_oracle(gus[j]), x16)
        g, u = ref[0][gate_rows], ref[0][gate_rows + 32]
        eg, eu = TOL * absum[0][gate_rows], TOL * absum[0][gate_rows + 32]
        want = xo.silu_mul(g, u)
        sil = g / (1.0 + np.exp(-g))
        bound = 1.1 * np.abs(u) * eg + np.abs(sil) * eu + 1.1 * eg * eu + 2.0 ** -10 * np.abs(want) + 1e-30
        assert np.all(np.abs(hg[j] - want) <= bound), float((np.abs(hg[j] - want) / bound).max())

    # stage 2 on the GPU's own h (as fp16, the down projection's input type)
    h16 = h.to(torch.float16).contiguous()
    wts = np.random.default_rng(2400).random(n).astype(np.float32)
    wts /= wts.sum()
    y = torch.full((n, hidden), float("nan"), dtype=dt, device="cuda")
    for _ in range(2):
        xfp.xfp_gemv_grouped_epilogue(dd, n, ptr([p.packed for p in pd]), ptr([h16[j] for j in range(n)]),
                                      ptr([y[j] for j in range(n)]), y_fp16, xfp.XFP_EPI_COMBINE,
                                      torch.from_numpy(wts).cuda(), wsd)
    torch.cuda.synchronize()
    h16_host = h16.view(torch.int16).cpu().numpy().view(np.uint16)
    want = np.zeros(hidden)
    bound = np.zeros(hidden)
    for j in range(n):
        ref, absum = xo.gemv(to_oracle(dns[j]), h16_host[j:j + 1])
        want += float(wts[j]) * ref[0]
        bound += abs(float(wts[j])) * absum[0]
    got = y[0].float().cpu().numpy().astype(np.float64)
    tol = TOL * bound + (2.0 ** -10 * np.abs(want) if y_fp16 else 0.0) + 1e-30
    assert np.all(np.abs(got - want) <= tol), float((np.abs(got - want) / tol).max())
    assert torch.isnan(y[1:].float()).all()          # only y[0] is written
    # the unfused path gives the same sums
    yu = torch.zeros((n, hidden), dtype=torch.float32, device="cuda")
    xfp.xfp_gemv_grouped(dd, n, ptr([p.packed for p in pd]), ptr([h16[j] for j in range(n)]),
                         ptr([yu[j] for j in range(n)]), False, wsd)
    torch.cuda.synchronize()
    plain = (yu.cpu().numpy().astype(np.float64) * wts[:, None].astype(np.float64)).sum(0)
    assert np.all(np.abs(got - plain) <= 0.05 * TOL * bound + (2.0 ** -10 * np.abs(want) if y_fp16 else 0.0) + 1e-30)


def test_fused_epilogues_are_refused_where_not_built():
    q = synth.random_quantized(0, 128, 256, 4, 0.0, seed=2500)      # V2 blobs have no fused store
    pm = xfp.pack_tensors(q)
    ptr = lambda ts: torch.tensor([t.data_ptr() for t in ts], dtype=torch.int64, device="cuda")
    x = _x_dev(synth.activations(1, 256, seed=1))
    y = torch.zeros(128, dtype=torch.float32, device="cuda")
    with pytest.raises(xfp.XfpError):
        xfp.xfp_gemv_grouped_epilogue(pm.desc, 1, ptr([pm.packed]), ptr([x]), ptr([y]), False, xfp.XFP_EPI_SWIGLU, None,
                                      pm.workspace)
    qa = synth.random_quantized(1, 96, 256, 3, 0.0, seed=2501)      # rows not a multiple of 64
    pa = xfp.pack_tensors(qa)
    with pytest.raises(xfp.XfpError):
        xfp.xfp_gemv_grouped_epilogue(pa.desc, 1, ptr([pa.packed]), ptr([x]), ptr([y]), False, xfp.XFP_EPI_SWIGLU, None,
                                      pa.workspace)
    with pytest.raises(xfp.XfpError):                                # the weighted sum needs its weights
        xfp.xfp_gemv_grouped_epilogue(pa.desc, 1, ptr([pa.packed]), ptr([x]), ptr([y]), False, xfp.XFP_EPI_COMBINE, None,
                                      pa.workspace)


def _bf16_x(batch, cols, seed):
    """N(0,1) activations rounded to bf16 (torch), with their exact values as doubles."""
    g = torch.Generator().manual_seed(seed)
    x = torch.randn((batch, cols), generator=g, dtype=torch.float32).to(torch.bfloat16)
    return x.cuda(), x.to(torch.float64).numpy()


@pytest.mark.parametrize("mode,bits", CASES)
@pytest.mark.parametrize("batch", [1, 2, 5, 16])
def test_bf16_activations_and_outputs(mode, bits, batch):
    """xfp_gemv_typed: bf16 x (converted to fp16 while staged) and y in fp32 / bf16 / fp16, every kernel the
    dispatcher can pick.  Reference: the oracle on the exact bf16 values.  Tolerance: the GEMV bound, plus
    2^-25 sum|W| for activations below 2^-14 (they land on the fp16 subnormal grid), plus the output rounding."""
    rows, cols = 288, 1152
    q = synth.random_quantized(mode, rows, cols, bits, 0.01, seed=2600 + 10 * mode + bits)
    pm = xfp.pack_tensors(q, col_bits=16)
    xd, x64 = _bf16_x(batch, cols, 2700 + batch)
    ref, absum = xo.gemv_x64(to_oracle(q), x64)
    tiny = 2.0 ** -25 * np.abs(xo.dequant(to_oracle(q)).view(np.float16).astype(np.float64)).sum(1)[None, :]
    for dt, ulp in ((torch.float32, 0.0), (torch.bfloat16, 2.0 ** -8), (torch.float16, 2.0 ** -11)):
        y = torch.full((batch, rows), float("nan"), dtype=dt, device="cuda")
        xfp.xfp_gemv_typed(pm.desc, pm.packed, xd, batch, y, pm.workspace)
        torch.cuda.synchronize()
        got = y.to(torch.float64).cpu().numpy()
        tol = TOL * absum + tiny + ulp * np.abs(ref) + 1e-30
        assert np.all(np.abs(got - ref) <= tol), (dt, float((np.abs(got - ref) / tol).max()))
    # fp16 x through the typed entry is the plain entry
    x16 = synth.activations(batch, cols, seed=2800)
    y1 = torch.empty((batch, rows), dtype=torch.float32, device="cuda")
    xfp.xfp_gemv_typed(pm.desc, pm.packed, _x_dev(x16), batch, y1, pm.workspace)
    y2 = pm.gemv(_x_dev(x16))
    torch.cuda.synchronize()
    assert torch.equal(y1, y2)


def test_bf16_activations_outside_the_fp16_range_are_clamped():
    q = synth.random_quantized(0, 64, 256, 4, 0.0, seed=2900)
    pm = xfp.pack_tensors(q)
    x = torch.zeros((1, 256), dtype=torch.bfloat16)
    x[0, 3], x[0, 100], x[0, 200] = 1.0e6, -3.0e38, 2.0 ** -30
    y = torch.empty((1, 64), dtype=torch.float32, device="cuda")
    xfp.xfp_gemv_typed(pm.desc, pm.packed, x.cuda(), 1, y, pm.workspace)
    torch.cuda.synchronize()
    xc = x.to(torch.float64).numpy().clip(-65504.0, 65504.0)
    xc[0, 200] = 0.0                                   # below half the smallest fp16 subnormal: rounds to zero
    ref, absum = xo.gemv_x64(to_oracle(q), xc)
    assert np.all(np.isfinite(y.cpu().numpy()))
    assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - ref) <= TOL * absum + 1e-30)


@pytest.mark.parametrize("mode,bits,batch", [(0, 4, 1), (0, 6, 4), (1, 3, 1), (1, 6, 1), (1, 6, 3), (1, 4, 8)])
def test_bf16_nan_and_tiny_activations_on_every_kernel(mode, bits, batch):
    """A NaN activation must poison y under bf16 as it does under fp16 (the clamp to the fp16 range applies to
    ordered values only), and bf16 values below 2^-14 are rounded to the fp16 subnormal grid by every kernel the
    dispatcher can pick -- the generic one (V2a at N = 6) included -- so the result does not depend on that pick."""
    rows, cols = 96, 512
    q = synth.random_quantized(mode, rows, cols, bits, 0.01, seed=2950 + 10 * mode + bits)
    pm = xfp.pack_tensors(q, col_bits=16)
    # tiny values only: exponents 2^-24 .. 2^-15, 8 significant bits
    rng = np.random.default_rng(2960 + bits)
    x64 = np.round(rng.uniform(1, 2, (batch, cols)) * 128) / 128 * 2.0 ** rng.integers(-24, -14, (batch, cols))
    x64 *= rng.choice([-1.0, 1.0], size=x64.shape)
    xb = torch.from_numpy(x64).to(torch.bfloat16)
    assert np.array_equal(xb.to(torch.float64).numpy(), x64)                   # exactly representable in bf16
    x_grid = xb.to(torch.float16).to(torch.float64).numpy()                    # what the fp16 conversion must give
    y = torch.empty((batch, rows), dtype=torch.float32, device="cuda")
    xfp.xfp_gemv_typed(pm.desc, pm.packed, xb.cuda(), batch, y, pm.workspace)
    torch.cuda.synchronize()
    ref, absum = xo.gemv_x64(to_oracle(q), x_grid)
    assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - ref) <= TOL * absum + 1e-30)
    # one NaN in batch row 0: every output of that row is NaN, the other rows stay finite
    xn = xb.clone()
    xn[0, 17] = float("nan")
    xfp.xfp_gemv_typed(pm.desc, pm.packed, xn.cuda(), batch, y, pm.workspace)
    torch.cuda.synchronize()
    got = y.cpu().numpy()
    assert np.all(np.isnan(got[0]))
    assert np.all(np.isfinite(got[1:]))


@pytest.mark.parametrize("bits,n,rows,cols", [(4, 3, 4096, 4096), (5, 3, 1024, 2048), (3, 2, 9600, 1024), (2, 7, 96, 512),
                                              (6, 4, 2080, 384)])
def test_grouped_v2_blobs_on_the_pair_kernel(bits, n, rows, cols):
    """Several V2 blobs of one shape in one launch (q, k and v of an attention block share x): blocks of all
    blobs are scheduled together, whole rounds first and K slices for the tail, every blob with its own
    codebooks and outlier slabs.  Sampled channels against the oracle, and the whole output against single calls."""
    qs = [synth.random_quantized(0, rows, cols, bits, 0.003 * (j + 1), seed=3000 + 7 * j + bits,
                                 placement="clustered" if j % 2 else "uniform") for j in range(n)]
    pms = [xfp.pack_tensors(q, col_bits=16) for q in qs]
    x16 = synth.activations(1, cols, seed=3100)
    xd = _x_dev(x16)
    desc = _group_desc(pms)
    ws = torch.zeros(n * xfp.xfp_packed_size(desc)[1], dtype=torch.uint8, device="cuda")
    ptr = lambda ts: torch.tensor([t.data_ptr() for t in ts], dtype=torch.int64, device="cuda")
    ys = torch.full((n, rows), float("nan"), dtype=torch.float32, device="cuda")
    for _ in range(2):      # twice: the split-K counters must come back to zero
        xfp.xfp_gemv_grouped(desc, n, ptr([p.packed for p in pms]), ptr([xd] * n), ptr([ys[j] for j in range(n)]), False, ws)
    torch.cuda.synchronize()
    rng = np.random.default_rng(3200)
    sample = np.unique(np.concatenate([rng.integers(0, rows, 48), [0, rows - 1, rows // 2]]))
    for j in range(n):
        got = ys[j].cpu().numpy().astype(np.float64)
        m = to_oracle(qs[j])
        for r in sample:
            ref, absum = xo.gemv(m, x16, int(r), int(r) + 1)
            assert abs(got[r] - ref[0, r]) <= TOL * absum[0, r] + 1e-30, (j, int(r))
        single = pms[j].gemv(xd)
        torch.cuda.synchronize()
        _, absum_all = (None, None)
        diff = np.abs(single[0].cpu().numpy().astype(np.float64) - got)
        scale = np.abs(got) + np.abs(single[0].cpu().numpy()) + 1e-6
        assert np.all(np.isfinite(got)) and np.all(diff <= 1e-3 * scale + 1e-4)


def _random_cases(count, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(count):
        mode = int(rng.integers(0, 2))
        bits = int(rng.integers(2, 7))
        rows = int(rng.choice([1, 7, 31, 32, 33, 63, 64, 65, 95, 160, 257, 416, 700, 1000, 2500, 4800, 9500]))
        cols = 128 * int(rng.choice([1, 2, 3, 5, 8, 11, 12, 13, 16, 24, 33]))
        batch = int(rng.choice([1, 1, 1, 2, 3, 4, 7, 8, 9, 16]))
        rate = float(rng.choice([0.0, 0.0005, 0.004, 0.02, 0.06]))
        placement = str(rng.choice(["uniform", "clustered", "one_row"]))
        ytype = str(rng.choice(["f32", "f16", "bf16"]))
        xtype = str(rng.choice(["f16", "f16", "bf16"]))
        cases.append((i, mode, bits, rows, cols, batch, rate, placement, xtype, ytype))
    return cases


@pytest.mark.parametrize("case", _random_cases(int(os.environ.get("XFP_SWEEP_CASES", "72")), 4242 + int(os.environ.get("XFP_SWEEP_SEED", "0"))),
                         ids=lambda c: "-".join(str(v) for v in c))
def test_randomized_shapes_types_and_outlier_structure(case):
    """A seeded sweep over everything the dispatcher keys on at once: mode, bit width, ragged channel counts
    (1 ... 9500: from a single row-block to more row-blocks than CTA slots), K from one to 33 super-chunks, batch 1..16, outlier rate and placement (including all outliers in one
    channel), activation and output types."""
    i, mode, bits, rows, cols, batch, rate, placement, xtype, ytype = case
    q = synth.random_quantized(mode, rows, cols, bits, rate, seed=5000 + i, placement=placement)
    pm = xfp.pack_tensors(q, col_bits=16 if i % 2 else 32)
    _check_dequant(q, pm)
    m = to_oracle(q)
    if xtype == "bf16":
        xd, x64 = _bf16_x(batch, cols, 6000 + i)
    else:
        x16 = synth.activations(batch, cols, seed=6000 + i)
        xd, x64 = _x_dev(x16), x16.view(np.float16).astype(np.float64)
    ref, absum = xo.gemv_x64(m, x64)
    dt = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}[ytype]
    ulp = {"f32": 0.0, "f16": 2.0 ** -11, "bf16": 2.0 ** -8}[ytype]
    y = torch.full((batch, rows), float("nan"), dtype=dt, device="cuda")
    for _ in range(2):
        xfp.xfp_gemv_typed(pm.desc, pm.packed, xd, batch, y, pm.workspace)
    torch.cuda.synchronize()
    got = y.to(torch.float64).cpu().numpy()
    tiny = 2.0 ** -25 * np.abs(xo.dequant(m).view(np.float16).astype(np.float64)).sum(1)[None, :] if xtype == "bf16" else 0.0
    tol = TOL * absum + tiny + ulp * np.abs(ref) + 1e-30
    assert np.all(np.isfinite(got))
    assert np.all(np.abs(got - ref) <= tol), float((np.abs(got - ref) / tol).max())


@pytest.mark.parametrize("mode,bits", [(1, 3), (1, 4), (0, 4), (0, 5), (1, 6)])
def test_grouped_typed_bf16(mode, bits):
    """The grouped launch with bf16 activations and outputs: plain for every mode (pair kernel, V2a kernels, generic),
    and the fused expert block (SiLU(gate)*up, then the weighted sum) where it exists."""
    n, rows_gu, hidden = 4, 256, 384
    inter = rows_gu // 2
    gus = [synth.random_quantized(mode, rows_gu, hidden, bits, 0.003, seed=3300 + j) for j in range(n)]
    if mode == 1:
        for q in gus[1:]:
            q.codebook = gus[0].codebook
    pg = [xfp.pack_tensors(q, col_bits=16) for q in gus]
    xd, x64 = _bf16_x(1, hidden, 3400)
    ptr = lambda ts: torch.tensor([t.data_ptr() for t in ts], dtype=torch.int64, device="cuda")
    dg = _group_desc(pg)
    wsg = torch.zeros(n * xfp.xfp_packed_size(dg)[1], dtype=torch.uint8, device="cuda")
    y = torch.full((n, rows_gu), float("nan"), dtype=torch.bfloat16, device="cuda")
    xfp.xfp_gemv_grouped_typed(dg, n, ptr([p.packed for p in pg]), ptr([xd] * n), torch.bfloat16, ptr([y[j] for j in range(n)]),
                               torch.bfloat16, xfp.XFP_EPI_NONE, None, wsg)
    torch.cuda.synchronize()
    refs = []
    for j in range(n):
        ref, absum = xo.gemv_x64(to_oracle(gus[j]), x64)
        refs.append((ref[0], absum[0]))
        tiny = 2.0 ** -25 * np.abs(xo.dequant(to_oracle(gus[j])).view(np.float16).astype(np.float64)).sum(1)
        got = y[j].to(torch.float64).cpu().numpy()
        assert np.all(np.abs(got - ref[0]) <= TOL * absum[0] + tiny + 2.0 ** -8 * np.abs(ref[0]) + 1e-30), j
    if mode == 0 or bits > 5:
        return          # fused stores exist for V2a up to N = 5
    h = torch.full((n, inter), float("nan"), dtype=torch.bfloat16, device="cuda")
    xfp.xfp_gemv_grouped_typed(dg, n, ptr([p.packed for p in pg]), ptr([xd] * n), torch.bfloat16, ptr([h[j] for j in range(n)]),
                               torch.bfloat16, xfp.XFP_EPI_SWIGLU, None, wsg)
    torch.cuda.synchronize()
    blocks = rows_gu // 64
    gate_rows = (np.arange(blocks)[:, None] * 64 + np.arange(32)[None, :]).reshape(-1)
    for j in range(n):
        ref, absum = refs[j]
        g, u = ref[gate_rows], ref[gate_rows + 32]
        eg, eu = TOL * absum[gate_rows] + 1e-9, TOL * absum[gate_rows + 32] + 1e-9
        want = xo.silu_mul(g, u)
        sil = g / (1.0 + np.exp(-g))
        bound = 1.1 * np.abs(u) * eg + np.abs(sil) * eu + 1.1 * eg * eu + 2.0 ** -7 * np.abs(want) + 1e-30
        assert np.all(np.abs(h[j].to(torch.float64).cpu().numpy() - want) <= bound), j
    dns = [synth.random_quantized(1, hidden, inter, bits, 0.003, seed=3500 + j) for j in range(n)]
    for q in dns[1:]:
        q.codebook = dns[0].codebook
    pd = [xfp.pack_tensors(q, col_bits=16) for q in dns]
    dd = _group_desc(pd)
    wsd = torch.zeros(n * xfp.xfp_packed_size(dd)[1], dtype=torch.uint8, device="cuda")
    wts = torch.tensor([0.4, 0.3, 0.2, 0.1], dtype=torch.float32, device="cuda")
    out = torch.full((1, hidden), float("nan"), dtype=torch.bfloat16, device="cuda")
    xfp.xfp_gemv_grouped_typed(dd, n, ptr([p.packed for p in pd]), ptr([h[j] for j in range(n)]), torch.bfloat16,
                               ptr([out[0]] * n), torch.bfloat16, xfp.XFP_EPI_COMBINE, wts, wsd)
    torch.cuda.synchronize()
    want = np.zeros(hidden)
    bound = np.zeros(hidden)
    for j in range(n):
        ref, absum = xo.gemv_x64(to_oracle(dns[j]), h[j:j + 1].to(torch.float64).cpu().numpy())
        want += float(wts[j]) * ref[0]
        bound += float(wts[j]) * absum[0]
    got = out[0].to(torch.float64).cpu().numpy()
    assert np.all(np.abs(got - want) <= TOL * bound + 2.0 ** -8 * np.abs(want) + 1e-6)
