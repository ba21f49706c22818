"""GPU parity: every C-ABI call against the CPU checker on the same seeded inputs.
Bit-exact for bits, order, outlier lists, codes and packed words; the statistic within 1e-5
relative (fp32 partial sums over at most 32 rows, fp64 above); centroids within 1e-4 relative
(expected equal bit for bit while no channel is flagged as inexact)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_13056_b200 import binding as B
from paper_2410_13056_b200 import inputs

import gpu_util as G

pytestmark = pytest.mark.gpu

STAT_RTOL = 1e-5
LUT_RTOL = 1e-4


@pytest.fixture(params=["ordered", "all_pairs"])
def assignment(request):
    """Runs a K-means test once per assignment method of the library; both must match the checker."""
    B.cmpq_set_lloyd_assignment(B.ASSIGN_ALL_PAIRS if request.param == "all_pairs" else B.ASSIGN_ORDERED)
    yield request.param
    B.cmpq_set_lloyd_assignment(B.ASSIGN_ORDERED)


def _lut_close(got, ref, W_absmax):
    np.testing.assert_allclose(got, ref, rtol=LUT_RTOL, atol=LUT_RTOL * W_absmax * 1e-3)


# ----------------------------------------------------------------------------- statistic
@pytest.mark.parametrize("dtype", [inputs.F16, inputs.BF16])
@pytest.mark.parametrize("n,d_in", [(512, 512), (1000, 264), (37, 1544), (3000, 4096), (1, 8), (9, 2056)])
def test_stats_vector_path(dtype, n, d_in):
    X = inputs.make_activations(n, d_in, dtype, 5, device="cuda", n_outlier_channels=3)
    sumsq, a = G.gpu_stats(X)
    ref = oracle.finalize_stats(oracle.collect_stats(inputs.as_u16(X), dtype))
    np.testing.assert_allclose(a, ref, rtol=STAT_RTOL)
    assert np.array_equal(a, np.sqrt(sumsq).astype(np.float32))


@pytest.mark.parametrize("dtype", [inputs.F16, inputs.BF16])
def test_stats_ragged_strided_and_chunked(dtype):
    # d_in not a multiple of 8 -> scalar path; a column slice of a wider matrix -> ldx > d_in
    X = inputs.make_activations(777, 301, dtype, 6, device="cuda")
    _, a = G.gpu_stats(X)
    ref = oracle.finalize_stats(oracle.collect_stats(inputs.as_u16(X), dtype))
    np.testing.assert_allclose(a, ref, rtol=STAT_RTOL)
    Xw = inputs.make_activations(500, 640, dtype, 7, device="cuda")
    for view in (Xw[:, 64:576], Xw[:, 3:260]):          # aligned slice, misaligned slice
        _, a = G.gpu_stats(view)
        ref = oracle.finalize_stats(oracle.collect_stats(inputs.as_u16(view.contiguous()), dtype))
        np.testing.assert_allclose(a, ref, rtol=STAT_RTOL)
    # accumulation over three chunks of tokens, one of them empty
    s1, a1 = G.gpu_stats(Xw, chunks=1)
    s3, a3 = G.gpu_stats(Xw, chunks=3)
    np.testing.assert_allclose(s3, s1, rtol=1e-6)
    sumsq = torch.ones(640, dtype=torch.float64, device="cuda")
    B.cmpq_collect_stats(Xw[:0], sumsq, B.workspace(B.OP_COLLECT_STATS, 640))
    assert torch.all(sumsq == 1.0)


def test_stats_closed_forms_and_determinism():
    X = torch.zeros(4096, 512, dtype=torch.bfloat16, device="cuda")
    X[:, 0] = 1.5
    X[100, 1] = -3.0
    X[:, 2] = 2.0 ** -20
    _, a = G.gpu_stats(X)
    assert a[0] == np.float32(1.5 * 64) and a[1] == 3.0 and a[2] == np.float32(2.0 ** -20 * 64) and a[3] == 0
    Y = inputs.make_activations(5000, 1024, inputs.BF16, 8, device="cuda")
    s1, _ = G.gpu_stats(Y)
    s2, _ = G.gpu_stats(Y)
    assert np.array_equal(s1, s2)


# ----------------------------------------------------------------------------- Algorithm 1
@pytest.mark.parametrize("d_in", [1, 5, 512, 4096, 11008, 28672])
@pytest.mark.parametrize("b", [2.0, 2.2, 2.5, 3.0, 3.7, 4.0])
def test_allocation_bit_exact(d_in, b):
    rng = np.random.default_rng(d_in + int(b * 10))
    a = np.exp(rng.standard_normal(d_in)).astype(np.float32)
    a[rng.integers(0, d_in, d_in // 7)] = a[0]            # ties
    for mode in (B.ALLOC_RANK, B.ALLOC_QUANTILE):
        bits, order = G.gpu_allocate(a, b, mode)
        rbits, rorder = oracle.allocate_bits(a, b, mode)
        assert np.array_equal(order, rorder)
        assert np.array_equal(bits, rbits)
    bits, _ = G.gpu_allocate(a, b, want_order=False)
    assert np.array_equal(bits, oracle.allocate_bits(a, b)[0])


# ----------------------------------------------------------------------------- K-means, outliers
def _case(d_in, d_out, dtype, seed, b):
    W = inputs.make_weight(d_in, d_out, dtype, seed, device="cuda")
    rng = np.random.default_rng(seed)
    a = np.exp(rng.standard_normal(d_in)).astype(np.float32)
    bits, _ = oracle.allocate_bits(a, b)
    return W, inputs.as_u16(W), a, bits


@pytest.mark.parametrize("dtype", [inputs.F16, inputs.BF16])
@pytest.mark.parametrize("d_in,d_out,T", [(96, 512, 10), (40, 1000, 6), (24, 4096, 20), (12, 11008, 5),
                                          (6, 28672, 4), (50, 37, 12), (64, 16, 30), (9, 1, 3), (5, 32768, 2)])
def test_quantize_layer_matches_checker(dtype, d_in, d_out, T, assignment):
    W, Wu, a, bits = _case(d_in, d_out, dtype, 21 + d_out, 3.0)
    bits[: d_in // 3] = 2
    bits[d_in // 3: 2 * d_in // 3] = 4
    rng = np.random.default_rng(d_out)
    nnz = min(d_in * d_out // 50, 500)
    lin = np.sort(rng.choice(d_in * d_out, nnz, replace=False))
    rows, cols = (lin // d_out).astype(np.int32), (lin % d_out).astype(np.int32)
    lut, codes, inexact, sweeps = G.gpu_quantize(W, bits, rows, cols, T)
    rlut, rcodes = oracle.quantize_layer(Wu, dtype, bits, rows, cols, T)
    assert inexact == 0
    assert np.array_equal(codes, rcodes)
    assert np.array_equal(lut.view(np.uint32), rlut.view(np.uint32))   # stronger than LUT_RTOL
    _lut_close(lut, rlut, 8.0)
    assert 0 < sweeps <= (T + 1) * d_out * int((1 << bits.astype(np.int64)).sum())


def test_quantize_layer_degenerate_channels(assignment):
    d_out = 256
    rows_ = []
    rows_.append(np.zeros(d_out))                                       # all zero
    rows_.append(np.full(d_out, 0.375))                                 # constant
    rows_.append(np.where(np.arange(d_out) % 8 == 0, -3.0, 1.0))        # two values
    z = np.zeros(d_out); z[::2] = -0.0; rows_.append(z)                 # signed zeros
    r = np.zeros(d_out); r[:5] = [1, 2, 3, 4, 5]; rows_.append(r)       # mass on one value -> duplicate starts
    rows_.append(np.linspace(-1, 1, d_out))
    rows_.append(np.arange(d_out) % 3 - 1.0)                            # three values
    Wt = torch.tensor(np.stack(rows_), dtype=torch.float16).cuda()
    Wu = inputs.as_u16(Wt)
    none = np.zeros(0, np.int32)
    for c in (2, 3, 4):
        for T in (0, 1, 3, 25):
            bits = np.full(len(rows_), c, np.uint8)
            lut, codes, inexact, _ = G.gpu_quantize(Wt, bits, none, none, T)
            rlut, rcodes = oracle.quantize_layer(Wu, inputs.F16, bits, none, none, T)
            assert np.array_equal(codes, rcodes), (c, T)
            assert np.array_equal(lut.view(np.uint32), rlut.view(np.uint32)), (c, T)


def test_wide_dynamic_range_is_flagged_not_hidden(assignment):
    d_out = 512
    x = np.random.default_rng(0).standard_normal((4, d_out)).astype(np.float32)
    x[1, 0] = 2.0 ** 60
    x[1, 1] = 2.0 ** -60
    Wt = torch.tensor(x, dtype=torch.bfloat16).cuda()
    bits = np.full(4, 3, np.uint8)
    none = np.zeros(0, np.int32)
    lut, codes, inexact, _ = G.gpu_quantize(Wt, bits, none, none, 10)
    assert inexact == 1
    rlut, rcodes = oracle.quantize_layer(inputs.as_u16(Wt), inputs.BF16, bits, none, none, 10)
    np.testing.assert_allclose(lut, rlut, rtol=LUT_RTOL)
    # whatever the summation order did to the flagged channel's centroids, the codes must be the
    # first-minimum codes of the centroids the library itself returned
    xw = Wt.float().cpu().numpy()
    xw = np.where(xw == 0, np.float32(0), xw)
    for i in range(4):
        d = np.abs(xw[i][:, None] - lut[i][None, :8]).astype(np.float32)
        assert np.array_equal(codes[i], np.argmin(d, axis=1)), i
    for i in (0, 2, 3):   # the other channels are exact: same bytes as the checker
        assert np.array_equal(codes[i], rcodes[i]) and np.array_equal(lut[i].view(np.uint32), rlut[i].view(np.uint32))


@pytest.mark.parametrize("dtype", [inputs.F16, inputs.BF16])
@pytest.mark.parametrize("d_in,d_out,n_act,n_q,T", [(64, 512, 2, 40, 8), (48, 1000, 0, 77, 5), (40, 300, 3, 0, 5),
                                                    (33, 4096, 1, 500, 10), (20, 64, 0, 0, 3), (16, 11008, 1, 88, 4),
                                                    (10, 50, 2, 8 * 50, 4)])
def test_extract_outliers_bit_exact(dtype, d_in, d_out, n_act, n_q, T, assignment):
    W, Wu, a, bits = _case(d_in, d_out, dtype, 77 + d_in, 2.5)
    rows, cols, vals = G.gpu_extract(W, a, bits, n_act, n_q, T)
    rr, rc, rv = oracle.extract_outliers(Wu, dtype, a, bits, n_act, n_q, T)
    assert np.array_equal(rows, rr) and np.array_equal(cols, rc) and np.array_equal(vals, rv)


def test_extract_outliers_ties_across_rows(assignment):
    d_in, d_out = 12, 128
    base = (np.linspace(-1, 1, d_out) ** 3).astype(np.float16)
    Wt = torch.from_numpy(np.tile(base, (d_in, 1))).cuda()
    a = np.arange(d_in, dtype=np.float32)
    bits = np.full(d_in, 2, np.uint8)
    for n_q in (1, 7, 11, 12, 30):
        got = G.gpu_extract(Wt, a, bits, 1, n_q, 4)
        ref = oracle.extract_outliers(inputs.as_u16(Wt), inputs.F16, a, bits, 1, n_q, 4)
        for g, r in zip(got, ref):
            assert np.array_equal(g, r), n_q


# ----------------------------------------------------------------------------- packing
@pytest.mark.parametrize("d_in,d_out", [(23, 1), (23, 31), (23, 32), (23, 33), (40, 100), (16, 4096), (9, 11008),
                                        (300, 512), (7, 28672), (5, 1000)])
def test_pack_bit_exact(d_in, d_out):
    rng = np.random.default_rng(d_in * d_out)
    bits = rng.integers(2, 5, d_in).astype(np.uint8)
    codes = (rng.integers(0, 16, (d_in, d_out)) & ((1 << bits[:, None]) - 1)).astype(np.uint8)
    got = G.gpu_pack(codes, bits)
    ref = oracle.pack(codes, bits)
    for g, r, name in zip(got, ref, ("packed", "row_off", "perm", "seg_rows")):
        assert np.array_equal(g, r), name
    for only in (2, 3, 4):                                   # single-width layers leave segments empty
        b1 = np.full(d_in, only, np.uint8)
        c1 = codes & ((1 << only) - 1)
        for g, r in zip(G.gpu_pack(c1, b1), oracle.pack(c1, b1)):
            assert np.array_equal(g, r)


# ----------------------------------------------------------------------------- timing aid
def test_phase_events_bracket_the_three_kernels_once():
    W, Wu, a, bits = _case(64, 2048, inputs.BF16, 5, 3.0)
    none = np.zeros(0, np.int32)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    B.cmpq_lloyd_phase_events(ev)
    lut1, codes1, _, _ = G.gpu_quantize(W, bits, none, none, 6)
    torch.cuda.synchronize()
    spans = [ev[i].elapsed_time(ev[i + 1]) for i in range(3)]
    assert all(s > 0 for s in spans)
    # the hook is consumed by one call; a second call is neither timed nor changed by it
    lut2, codes2, _, _ = G.gpu_quantize(W, bits, none, none, 6)
    assert np.array_equal(codes1, codes2) and np.array_equal(lut1, lut2)
    B.cmpq_lloyd_phase_events(ev)
    B.cmpq_lloyd_phase_events(None)   # cancel
    with pytest.raises(B.CmpqError):
        B._check(B.lib().cmpq_lloyd_phase_events(1, None, None, None), "cmpq_lloyd_phase_events")


# ----------------------------------------------------------------------------- value tables: less common shapes
def _log_uniform(d_in, d_out, lo_exp, hi_exp, seed, tdt):
    """Weights with magnitudes spread evenly over many binades and both signs: many distinct 16-bit
    values and many occupied high bytes, unlike Gaussian-like weights."""
    rng = np.random.default_rng(seed)
    mag = np.exp2(rng.uniform(lo_exp, hi_exp, (d_in, d_out)))
    sign = np.where(rng.random((d_in, d_out)) < 0.5, -1.0, 1.0)
    return torch.tensor(mag * sign, dtype=torch.float32).to(tdt).cuda()


@pytest.mark.parametrize("dtype,tdt,d_in,d_out,lo,hi", [
    (inputs.BF16, torch.bfloat16, 12, 768, -20, 13),     # more than 32 occupied high bytes: several table passes
    (inputs.BF16, torch.bfloat16, 3, 32768, -9, 3),      # more distinct values than a warp stages in shared memory
    (inputs.F16, torch.float16, 6, 8192, -14, 3),        # fp16: both at once
])
def test_quantize_layer_wide_value_tables(dtype, tdt, d_in, d_out, lo, hi, assignment):
    W = _log_uniform(d_in, d_out, lo, hi, 3 + d_out, tdt)
    Wu = inputs.as_u16(W)
    bits = np.array([2, 3, 4] * d_in, np.uint8)[:d_in]
    none = np.zeros(0, np.int32)
    assert max(len(np.unique(r)) for r in Wu) > 600   # the shapes above rely on many distinct values
    lut, codes, inexact, _ = G.gpu_quantize(W, bits, none, none, 9)
    rlut, rcodes = oracle.quantize_layer(Wu, dtype, bits, none, none, 9)
    assert inexact == 0
    assert np.array_equal(codes, rcodes)
    assert np.array_equal(lut.view(np.uint32), rlut.view(np.uint32))


@pytest.mark.parametrize("per_row", [1, 15, 16, 17, 40])
def test_quantize_layer_removed_positions_list_and_bitmap(per_row, assignment):
    d_in, d_out, T = 10, 2048, 7
    W, Wu, a, bits = _case(d_in, d_out, inputs.BF16, 99, 3.0)
    rng = np.random.default_rng(per_row)
    lin = np.sort(np.concatenate([i * d_out + rng.choice(d_out, per_row, replace=False) for i in range(d_in)]))
    rows, cols = (lin // d_out).astype(np.int32), (lin % d_out).astype(np.int32)
    lut, codes, inexact, _ = G.gpu_quantize(W, bits, rows, cols, T)
    rlut, rcodes = oracle.quantize_layer(Wu, inputs.BF16, bits, rows, cols, T)
    assert np.array_equal(codes, rcodes)
    assert np.array_equal(lut.view(np.uint32), rlut.view(np.uint32))


def test_extract_outliers_wide_value_tables(assignment):
    d_in, d_out = 9, 4096
    W = _log_uniform(d_in, d_out, -12, 2, 17, torch.float16)
    a = np.arange(d_in, dtype=np.float32)[::-1].copy()
    bits = np.array([2, 3, 4] * 3, np.uint8)
    got = G.gpu_extract(W, a, bits, 1, 300, 6)
    ref = oracle.extract_outliers(inputs.as_u16(W), inputs.F16, a, bits, 1, 300, 6)
    for g, r in zip(got, ref):
        assert np.array_equal(g, r)


# ----------------------------------------------------------------------------- fused protection + final fit
@pytest.mark.parametrize("dtype", [inputs.F16, inputs.BF16])
@pytest.mark.parametrize("d_in,d_out,n_act,n_q,T", [(64, 512, 2, 40, 8), (33, 4096, 1, 500, 10), (20, 64, 0, 0, 3),
                                                    (6, 1024, 1, 900, 5), (10, 50, 2, 8 * 50, 4), (40, 300, 3, 0, 5),
                                                    (5, 1, 1, 2, 3)])
def test_protect_and_quantize_equals_the_two_calls(dtype, d_in, d_out, n_act, n_q, T, assignment):
    W, Wu, a, bits = _case(d_in, d_out, dtype, 55 + d_in, 2.8)
    bits[::3] = 4
    rows, cols, vals = G.gpu_extract(W, a, bits, n_act, n_q, T)
    lut, codes, inexact, sweeps = G.gpu_quantize(W, bits, rows, cols, T)
    nnz = n_act * d_out + n_q
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
    r2 = torch.full((max(nnz, 1),), -1, dtype=torch.int32, device="cuda")
    c2 = torch.full((max(nnz, 1),), -1, dtype=torch.int32, device="cuda")
    v2 = torch.zeros(max(nnz, 1), dtype=torch.int16, device="cuda")
    lut2 = torch.full((d_in, 16), -7.0, dtype=torch.float32, device="cuda")
    codes2 = torch.full((d_in, d_out), 255, dtype=torch.uint8, device="cuda")
    counters = torch.zeros(2, dtype=torch.int64, device="cuda")
    B.cmpq_protect_and_quantize(W, dev(a), dev(bits), n_act, n_q, T, r2[:nnz], c2[:nnz], v2[:nnz], lut2, codes2,
                                B.workspace(B.OP_PROTECT_AND_QUANTIZE, d_in, d_out),
                                inexact_rows=counters[0:1].view(torch.int32)[0:1], sweeps=counters[1:2])
    torch.cuda.synchronize()
    assert np.array_equal(r2[:nnz].cpu().numpy(), rows) and np.array_equal(c2[:nnz].cpu().numpy(), cols)
    assert np.array_equal(v2[:nnz].cpu().numpy().view(np.uint16), vals)
    assert np.array_equal(codes2.cpu().numpy(), codes)
    assert np.array_equal(lut2.cpu().numpy().view(np.uint32), lut.view(np.uint32))
    c = counters.cpu().numpy()
    assert int(c[0] & 0xffffffff) == inexact and int(c[1]) == sweeps
    # and against the checker
    rlut, rcodes = oracle.quantize_layer(Wu, dtype, bits, rows, cols, T)
    assert np.array_equal(codes2.cpu().numpy(), rcodes)


# ----------------------------------------------------------------------------- layout conversion
@pytest.mark.parametrize("shape", [(1, 1), (64, 64), (65, 63), (300, 1030), (66, 2), (8, 200), (72, 136), (4096, 11008),
                                   (11008, 4096)])
# leading dimensions that are multiples of 8 (with extents that are): 128-bit accesses; even: 32-bit; odd: element-wise
@pytest.mark.parametrize("pads", [(8, 16), (4, 6), (3, 5)])
@pytest.mark.parametrize("tdt", [torch.float16, torch.bfloat16])
def test_transpose16_is_the_transpose(shape, pads, tdt):
    """Plain definition: dst[c][r] = src[r][c], raw 16-bit patterns (checked against numpy on the host)."""
    g = torch.Generator(device="cuda")
    g.manual_seed(shape[0] * 7 + shape[1])
    bits = torch.randint(-32768, 32768, shape, dtype=torch.int16, device="cuda", generator=g)
    src = bits.view(tdt)
    full = torch.full((shape[1], shape[0] + pads[0]), 1.0, dtype=tdt, device="cuda")
    dst = full[:, : shape[0]]                                                               # padded rows
    B.cmpq_transpose16(src, dst)
    wide = torch.full((shape[0], shape[1] + pads[1]), 1.0, dtype=tdt, device="cuda")
    wide[:, : shape[1]] = src
    dst2 = torch.empty((shape[1], shape[0]), dtype=tdt, device="cuda")
    B.cmpq_transpose16(wide[:, : shape[1]], dst2)                                            # padded source
    torch.cuda.synchronize()
    ref = np.ascontiguousarray(bits.cpu().numpy().T)
    assert np.array_equal(dst.contiguous().view(torch.int16).cpu().numpy(), ref)
    assert np.array_equal(dst2.view(torch.int16).cpu().numpy(), ref)
    assert torch.all(full[:, shape[0]:] == 1.0)                                             # padding untouched
