"""Pins for the oracle's outlier protection (Section 3.2.2), final quantization, packing
(Section 5.1 accounting) and reconstruction error (dY = X (W - What)).  CPU only."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2410_13056_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _layer(d_in=48, d_out=64, n=96, dtype=inputs.F16, seed=3):
    W = inputs.make_weight(d_in, d_out, dtype, seed)
    X = inputs.make_activations(n, d_in, dtype, seed, n_outlier_channels=3)
    return inputs.as_u16(X), inputs.as_u16(W), W, X


def _f32(t):
    return t.float().numpy()


# ----------------------------------------------------------------------------- outliers
@pytest.mark.parametrize("dtype", [inputs.F16, inputs.BF16])
@pytest.mark.parametrize("n_act,n_q", [(0, 0), (2, 0), (0, 9), (3, 17), (1, 200)])
def test_outlier_sets_against_full_sort(dtype, n_act, n_q):
    Xu, Wu, W, X = _layer(dtype=dtype)
    d_in, d_out = Wu.shape
    a = oracle.finalize_stats(oracle.collect_stats(Xu, dtype))
    bits, order = oracle.allocate_bits(a, 3.0)
    T = 6
    rows, cols, vals, lut1, err = oracle.extract_outliers(Wu, dtype, a, bits, n_act, n_q, T, want_fit=True)
    nnz = n_act * d_out + n_q
    assert rows.shape == (nnz,)
    lin = rows.astype(np.int64) * d_out + cols
    assert np.all(np.diff(lin) > 0)                              # strictly increasing (row, col)
    assert np.array_equal(vals, Wu[rows, cols])                  # original 16-bit patterns
    act_rows = np.sort(order[d_in - n_act:]) if n_act else np.zeros(0, np.int32)
    assert np.array_equal(act_rows, np.sort(np.argsort(a, kind="stable")[d_in - n_act:]))
    is_act = np.zeros(d_in, bool)
    is_act[act_rows] = True
    in_act = is_act[rows]
    assert in_act.sum() == n_act * d_out                         # whole rows
    # the provisional fit is the channel K-means of W' (act rows zeroed)
    Wf = _f32(W).copy()
    Wf[is_act] = 0
    for i in (0, d_in // 2, d_in - 1, int(act_rows[0]) if n_act else 1):
        l, c, e = oracle.lloyd(Wf[i], 1 << int(bits[i]), T)
        assert np.array_equal(l, lut1[i])
        if not is_act[i]:
            assert np.array_equal(e, err[i])
    # O_q = the n_q largest errors outside the act rows, ties by linear index (numpy lexsort)
    cand = np.flatnonzero(~np.repeat(is_act, d_out))
    e = err.reshape(-1)[cand]
    top = cand[np.lexsort((cand, -e.astype(np.float64)))[:n_q]]
    assert np.array_equal(np.sort(top), lin[~in_act])
    if n_q and n_q < cand.size:
        rest = np.setdiff1d(cand, top)
        assert err.reshape(-1)[rest].max() <= err.reshape(-1)[top].min()   # I5


def test_outlier_ties_resolve_by_linear_index():
    # every row identical -> every row has identical errors -> ties across rows
    d_in, d_out = 6, 32
    base = (np.linspace(-1, 1, d_out) ** 3).astype(np.float16)
    W = torch.from_numpy(np.tile(base, (d_in, 1)))
    Wu = inputs.as_u16(W)
    a = np.arange(d_in, dtype=np.float32)
    bits = np.full(d_in, 2, np.uint8)
    rows, cols, vals, lut1, err = oracle.extract_outliers(Wu, inputs.F16, a, bits, 1, 7, 4, want_fit=True)
    assert np.all(rows[-d_out:] == d_in - 1)        # act row = largest a
    q_rows, q_cols = rows[:-d_out], cols[:-d_out]
    assert all(np.array_equal(err[i], err[0]) for i in range(5))
    # walk the error levels downwards; inside a level lower rows (smaller linear index) go first
    want = []
    for level in np.unique(err[0])[::-1]:
        want += [(i, int(j)) for i in range(5) for j in np.flatnonzero(err[0] == level)]
    want = sorted(want[:7])
    got = sorted(zip(q_rows.tolist(), q_cols.tolist()))
    assert got == want
    per_row = np.bincount(q_rows, minlength=5)
    assert per_row.max() > per_row.min() and np.all(np.diff(per_row) <= 0)   # a level was cut between rows


def test_bad_counts_are_rejected():
    Xu, Wu, W, X = _layer()
    a = np.ones(Wu.shape[0], np.float32)
    bits = np.full(Wu.shape[0], 3, np.uint8)
    with pytest.raises(ValueError):
        oracle.extract_outliers(Wu, inputs.F16, a, bits, Wu.shape[0] + 1, 0, 2)
    with pytest.raises(ValueError):
        oracle.extract_outliers(Wu, inputs.F16, a, bits, 1, (Wu.shape[0] - 1) * Wu.shape[1] + 1, 2)


# ----------------------------------------------------------------------------- final quantization
@pytest.mark.parametrize("dtype", [inputs.F16, inputs.BF16])
def test_quantize_layer_zeroes_outliers_and_fits_each_channel(dtype):
    Xu, Wu, W, X = _layer(dtype=dtype)
    d_in, d_out = Wu.shape
    a = oracle.finalize_stats(oracle.collect_stats(Xu, dtype))
    bits, _ = oracle.allocate_bits(a, 2.5)
    rows, cols, vals = oracle.extract_outliers(Wu, dtype, a, bits, 2, 25, 5)
    lut, codes = oracle.quantize_layer(Wu, dtype, bits, rows, cols, 5)
    Wf = _f32(W).copy()
    Wf[rows, cols] = 0
    for i in range(d_in):
        l, c, _ = oracle.lloyd(Wf[i], 1 << int(bits[i]), 5)
        assert np.array_equal(l, lut[i]) and np.array_equal(c, codes[i])
        assert codes[i].max() < (1 << int(bits[i]))
    act = np.unique(rows[np.bincount(rows, minlength=d_in)[rows] == d_out])
    assert len(act) == 2 and np.all(lut[act] == 0) and np.all(codes[act] == 0)


def test_recon_error_matches_dense_float64_and_outliers_help():
    Xu, Wu, W, X = _layer(dtype=inputs.BF16, d_in=40, d_out=56, n=64)
    a = oracle.finalize_stats(oracle.collect_stats(Xu, inputs.BF16))
    bits, _ = oracle.allocate_bits(a, 3.0)
    E = []
    for n_act, n_q in [(0, 0), (2, 0), (2, 30)]:
        rows, cols, vals = oracle.extract_outliers(Wu, inputs.BF16, a, bits, n_act, n_q, 8)
        lut, codes = oracle.quantize_layer(Wu, inputs.BF16, bits, rows, cols, 8)
        What = np.take_along_axis(lut.astype(np.float64), codes.astype(np.int64), axis=1)
        O = np.zeros_like(What)
        O[rows, cols] = _f32(W)[rows, cols]
        ref = np.linalg.norm(X.double().numpy() @ (W.double().numpy() - What - O))
        got = oracle.recon_error(Xu, Wu, inputs.BF16, lut, codes, rows, cols, vals)
        assert got == pytest.approx(ref, rel=1e-12)
        E.append(got)
    assert E[0] > E[1] > E[2] > 0
    # channels with no more distinct values than centroids are reproduced exactly
    Wc = torch.from_numpy(np.tile(np.array([0.5, -0.25, 0.125, 1.0], np.float32), (40, 14))).to(torch.bfloat16)
    Wcu = inputs.as_u16(Wc)
    none = np.zeros(0, np.int32)
    lut, codes = oracle.quantize_layer(Wcu, inputs.BF16, np.full(40, 2, np.uint8), none, none, 4)
    assert oracle.recon_error(Xu, Wcu, inputs.BF16, lut, codes, none, none, np.zeros(0, np.uint16)) == 0.0


# ----------------------------------------------------------------------------- packing
def _pack_reference(codes, bits):
    """Independent route: numpy.packbits on the little-endian bit expansion of every code."""
    d_in, d_out = codes.shape
    words, perm, off = [], [], [0]
    for c in (2, 3, 4):
        for i in np.flatnonzero(bits == c):
            b = ((codes[i][:, None] >> np.arange(c)) & 1).astype(np.uint8).reshape(-1)
            b = np.concatenate([b, np.zeros((-len(b)) % 32, np.uint8)])
            w = np.packbits(b, bitorder="little").view("<u4")
            words.append(w)
            perm.append(i)
            off.append(off[-1] + len(w))
    return np.concatenate(words), np.array(off, np.int64), np.array(perm, np.int32)


@pytest.mark.parametrize("d_out", [1, 5, 16, 31, 32, 33, 64, 100, 257])
def test_pack_layout_round_trip_and_word_count(d_out):
    rng = np.random.default_rng(d_out)
    d_in = 23
    bits = rng.integers(2, 5, d_in).astype(np.uint8)
    codes = (rng.integers(0, 16, (d_in, d_out)) & ((1 << bits[:, None]) - 1)).astype(np.uint8)
    packed, row_off, perm, seg_rows = oracle.pack(codes, bits)
    ref_packed, ref_off, ref_perm = _pack_reference(codes, bits)
    assert np.array_equal(packed, ref_packed)
    assert np.array_equal(row_off, ref_off)
    assert np.array_equal(perm, ref_perm)
    assert np.array_equal(seg_rows, [(bits == c).sum() for c in (2, 3, 4)])
    assert len(packed) == sum(-(-d_out * int(c) // 32) for c in bits) == oracle.packed_words(bits, d_out)
    assert np.array_equal(oracle.unpack(packed, row_off, perm, bits, d_out), codes)   # I9
    if d_out % 32 == 0:
        assert len(packed) * 4 == d_out * int(bits.astype(np.int64).sum()) // 8


def test_worked_packing_example():
    # 3-bit channel, codes 1,2,3,4,5,6,7,0,1,2,3: stream LSB first; by hand:
    # word0 = sum code_j << 3j for j < 10 (30 bits) plus the low 2 bits of code 10 at bits 30,31
    codes = np.array([[1, 2, 3, 4, 5, 6, 7, 0, 1, 2, 3]], np.uint8)
    packed, row_off, perm, seg = oracle.pack(codes, np.array([3], np.uint8))
    w0 = sum(int(c) << (3 * j) for j, c in enumerate(codes[0][:10])) | ((3 & 3) << 30)
    assert packed.tolist() == [w0, 3 >> 2] and row_off.tolist() == [0, 2]
    # 2-bit then 4-bit channel order regardless of channel id
    codes = np.array([[15, 1], [3, 2]], np.uint8)
    packed, row_off, perm, seg = oracle.pack(codes, np.array([4, 2], np.uint8))
    assert perm.tolist() == [1, 0] and packed.tolist() == [3 | (2 << 2), 15 | (1 << 4)]
    assert seg.tolist() == [1, 0, 1]


def test_storage_overhead_values_printed_in_the_paper():
    for line in open(os.path.join(GOLD, "storage_overhead.txt")):
        if not line.strip() or line.startswith("#"):
            continue
        d_out, c, tag, lutb, rel, val = line.split()
        got = oracle.metadata_bits_per_weight(np.full(7, int(c), np.uint8), int(d_out), int(tag), int(lutb))
        if rel == "approx":
            assert round(got, 2) == float(val)
        else:
            assert got < float(val)
    assert oracle.metadata_bits_per_weight(np.full(7, 3, np.uint8), 4096) == (4 + 8 * 16) / 4096


# ----------------------------------------------------------------------------- whole pass
def test_layer_pass_is_the_composition_of_the_steps():
    Xu, Wu, W, X = _layer(dtype=inputs.F16, d_in=64, d_out=96, n=128)
    n_act, n_q = 2, 40
    out = oracle.layer_pass(Xu, Wu, inputs.F16, 3.0, n_act, n_q, 7)
    a = oracle.finalize_stats(oracle.collect_stats(Xu, inputs.F16))
    bits, _ = oracle.allocate_bits(a, 3.0)
    rows, cols, vals = oracle.extract_outliers(Wu, inputs.F16, a, bits, n_act, n_q, 7)
    lut, codes = oracle.quantize_layer(Wu, inputs.F16, bits, rows, cols, 7)
    packed, row_off, perm, seg = oracle.pack(codes, bits)
    for k, v in dict(a=a, bits=bits, rows=rows, cols=cols, vals=vals, lut=lut, codes=codes,
                     packed=packed, row_off=row_off, perm=perm, seg_rows=seg).items():
        assert np.array_equal(out[k], v), k
