"""Pins of the checker's stored table formats (Section 5.1 of the paper: tables in FP16, 16 bits per
centroid; variant with 4 bits per centroid) against things other than itself: numpy's float16
conversion, closed forms of a uniform grid, a channel worked by hand, the storage figures the paper
prints."""
import numpy as np
import pytest

import oracle


def test_float_to_half_matches_numpy_on_every_rounding_case():
    rng = np.random.default_rng(3)
    vals = [0.0, -0.0, 1.0, -1.0, 65504.0, 65519.99, 65520.0, 7e4, -7e4, 2.0 ** -14, 2.0 ** -24, 2.0 ** -25,
            2.0 ** -25 * 1.0001, 2.0 ** -26, 1.5 * 2.0 ** -24, 2.5 * 2.0 ** -24, np.inf, -np.inf]
    # ties between neighbouring binary16 values in several binades (exact halves: ties go to even)
    for e in (-14, -8, -1, 0, 3, 15):
        for m in (0, 1, 2, 511, 1022, 1023):
            lo = (1024 + m) * 2.0 ** (e - 10)
            vals += [lo, lo + 0.5 * 2.0 ** (e - 10), lo + 0.49999 * 2.0 ** (e - 10), lo + 0.50001 * 2.0 ** (e - 10)]
    v = np.concatenate([np.array(vals, np.float32),
                        (rng.standard_normal(4000) * 10.0 ** rng.uniform(-9, 5, 4000)).astype(np.float32)])
    with np.errstate(over="ignore"):
        ref = v.astype(np.float16).view(np.uint16)
    assert np.array_equal(oracle.float_to_half(v), ref)
    assert oracle.float_to_half(np.array([np.nan], np.float32))[0] & 0x7c00 == 0x7c00


def test_f16_tables_round_trip_and_zero_tail():
    rng = np.random.default_rng(4)
    bits = np.array([2, 3, 4, 3], np.uint8)
    lut = rng.normal(0, 0.02, (4, 16)).astype(np.float32)
    l16 = oracle.lut_to_f16(lut, bits)
    for i, c in enumerate(bits):
        K = 1 << int(c)
        assert np.array_equal(l16[i, :K], lut[i, :K].astype(np.float16).view(np.uint16))
        assert not l16[i, K:].any()
    back = oracle.lut_from_f16(l16)
    assert np.array_equal(back, l16.view(np.float16).astype(np.float32))
    # values already on the binary16 grid survive unchanged
    exact = back.copy()
    assert np.array_equal(oracle.lut_from_f16(oracle.lut_to_f16(exact, np.full(4, 4, np.uint8)))[:, :4], exact[:, :4])


def test_u4_hand_worked_channel():
    """Eight centroids between lo = -1 and hi = 2 (both binary16 values): the step is 0.2f and the codes
    follow by hand, (c + 1) / 0.2 rounded half to even."""
    bits = np.array([3], np.uint8)
    c = np.array([-1.0, -0.91, -0.7, -0.3, 0.0, 0.5, 1.29, 2.0], np.float32)
    lut = np.zeros((1, 16), np.float32)
    lut[0, :8] = c
    st = oracle.lut_to_u4(lut, bits)[0]
    codes = [(st[k >> 1] >> (4 * (k & 1))) & 15 for k in range(16)]
    # by hand: -1 -> 0;  -0.91 -> 0.45 -> 0;  0 -> 5;  1.29 -> 11.45 -> 11;  2 -> 15.  -0.7, -0.3 and 0.5 sit
    # on half steps in exact arithmetic; which way fp32 takes them is settled by numpy on the same quantities
    D = np.float32(np.float32(3.0) / np.float32(15.0))
    expect = [int(np.clip(np.rint(np.float32(np.float32(x) - np.float32(-1.0)) / D), 0, 15)) for x in c]
    assert codes[:8] == expect and codes[8:] == [0] * 8
    assert codes[0] == 0 and codes[4] == 5 and codes[6] == 11 and codes[7] == 15
    assert int(st[8]) | (int(st[9]) << 8) == 0xbc00 and int(st[10]) | (int(st[11]) << 8) == 0x4000   # -1.0 and 2.0 in binary16
    dec = oracle.lut_from_u4(st[None, :], bits)[0]
    assert np.array_equal(dec[:8], (np.float32(-1.0) + np.array(expect, np.float32) * D).astype(np.float32))
    assert not dec[8:].any()


@pytest.mark.parametrize("c", [2, 3, 4])
def test_u4_grid_properties(c):
    rng = np.random.default_rng(10 + c)
    d_in, K = 200, 1 << c
    bits = np.full(d_in, c, np.uint8)
    lut = np.zeros((d_in, 16), np.float32)
    lut[:, :K] = np.sort(rng.normal(0, 0.02, (d_in, K)).astype(np.float32), axis=1)
    lut[7, :K] = 0.125                         # a constant channel: zero step
    st = oracle.lut_to_u4(lut, bits)
    assert st.shape == (d_in, 12)
    dec = oracle.lut_from_u4(st, bits)
    lo16 = (st[:, 8].astype(np.uint16) | (st[:, 9].astype(np.uint16) << 8)).view(np.float16).astype(np.float32)
    hi16 = (st[:, 10].astype(np.uint16) | (st[:, 11].astype(np.uint16) << 8)).view(np.float16).astype(np.float32)
    assert np.array_equal(lo16, lut[:, 0].astype(np.float16).astype(np.float32))       # smallest / largest centroid,
    assert np.array_equal(hi16, lut[:, K - 1].astype(np.float16).astype(np.float32))   # rounded to binary16
    codes = np.stack([(st[:, k >> 1] >> (4 * (k & 1))) & 15 for k in range(16)], axis=1)
    assert np.all(np.diff(codes[:, :K].astype(int), axis=1) >= 0)                      # sorted centroids: sorted codes
    assert not codes[:, K:].any()
    step = (hi16 - lo16) / 15
    live = step > 0
    assert np.all(codes[live, 0] == 0) and np.all(codes[live, K - 1] == 15)            # the end points are the ends
    # half-step bound (plus the binary16 rounding of the two end points and fp32 rounding of the grid)
    err = np.abs(dec[:, :K] - lut[:, :K])
    bound = step[:, None] / 2 + np.abs(lut[:, [0]] - lo16[:, None]) + np.abs(lut[:, [K - 1]] - hi16[:, None]) + 1e-7
    assert np.all(err <= bound)
    assert not codes[7].any() and np.all(dec[7, :K] == np.float32(0.125))
    # independent route: numpy's rint on the same fp32 quantities
    t = (lut[:, :K] - lo16[:, None]).astype(np.float32)
    with np.errstate(divide="ignore", invalid="ignore"):
        ref = np.where(step[:, None] > 0, np.clip(np.rint((t / step[:, None].astype(np.float32)).astype(np.float32)), 0, 15), 0)
    assert np.array_equal(codes[:, :K], ref.astype(np.uint8))


def test_storage_figures_of_the_paper():
    """Section 5.1: one 4-bit tag and eight centroids per channel of 4096 weights cost about 0.03 bit per
    weight with FP16 tables and less than 0.01 with 4-bit tables; counting the two FP16 grid ends this
    build stores with the 4-bit codes gives 0.0166."""
    bits = np.full(4096, 3, np.uint8)
    f16 = oracle.metadata_bits_per_weight(bits, 4096, tag_bits=4, lut_bits=16)
    u4 = oracle.metadata_bits_per_weight(bits, 4096, tag_bits=4, lut_bits=4)
    assert f16 == (4 + 8 * 16) / 4096 and round(f16, 2) == 0.03
    assert u4 == (4 + 8 * 4) / 4096 and u4 < 0.01
    assert (4 + 8 * 4 + 2 * 16) / 4096 == pytest.approx(0.0166, abs=1e-4)
    # the stored arrays have exactly these sizes
    lut = np.zeros((4096, 16), np.float32)
    assert oracle.lut_to_f16(lut, bits)[:, :8].nbytes * 8 / (4096 * 4096) == 8 * 16 / 4096
    assert oracle.lut_to_u4(lut, bits).nbytes * 8 / (4096 * 4096) == pytest.approx((16 * 4 + 32) / 4096)
