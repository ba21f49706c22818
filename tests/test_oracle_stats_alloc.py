"""Pins for the oracle's statistic (Section 3.2.1) and Algorithm 1: closed forms, invariants,
library routines and the facts the paper prints.  CPU only."""
import os

import numpy as np
import pytest
import torch

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _facts():
    out = {}
    for line in open(os.path.join(GOLD, "allocation_facts.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            out[k] = float(v)
    return out


def _u16(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


# ----------------------------------------------------------------------------- widening
@pytest.mark.parametrize("dtype,tdt", [(oracle.F16, torch.float16), (oracle.BF16, torch.bfloat16)])
def test_widen_matches_torch_on_all_finite_patterns(dtype, tdt):
    pat = np.arange(0, 65536, 7, dtype=np.uint16)  # subnormals, normals, both signs
    ref = torch.from_numpy(pat.view(np.int16)).view(tdt).float().numpy()
    got = oracle.widen(pat, dtype)
    fin = np.isfinite(ref)
    assert np.array_equal(got[fin].view(np.uint32), ref[fin].view(np.uint32))
    assert np.all(~np.isfinite(got[~fin]))


# ----------------------------------------------------------------------------- statistic
@pytest.mark.parametrize("dtype,tdt", [(oracle.F16, torch.float16), (oracle.BF16, torch.bfloat16)])
def test_stats_constant_and_onehot_columns(dtype, tdt):
    n, d = 64, 5
    X = torch.zeros(n, d, dtype=tdt)
    X[:, 0] = 1.5          # constant column: |v| sqrt(n)
    X[:, 1] = -0.25
    X[17, 2] = 3.0         # one-hot column: |v|
    X[:, 4] = 2.0 ** -10   # small constant
    a = oracle.finalize_stats(oracle.collect_stats(_u16(X), dtype))
    assert a[0] == np.float32(1.5 * 8.0)
    assert a[1] == np.float32(0.25 * 8.0)
    assert a[2] == np.float32(3.0)
    assert a[3] == 0.0
    assert a[4] == np.float32(2.0 ** -10 * 8.0)


def test_stats_matches_numpy_norm_and_scales_exactly_by_powers_of_two():
    g = torch.Generator().manual_seed(1)
    X = (torch.randn(300, 37, generator=g) * torch.exp(torch.randn(37, generator=g))).to(torch.bfloat16)
    a = oracle.finalize_stats(oracle.collect_stats(_u16(X), oracle.BF16))
    ref = np.linalg.norm(X.double().numpy(), axis=0)
    np.testing.assert_allclose(a, ref, rtol=2e-7)
    X4 = (X.float() * 4.0).to(torch.bfloat16)  # exact in bf16
    a4 = oracle.finalize_stats(oracle.collect_stats(_u16(X4), oracle.BF16))
    assert np.array_equal(a4, a * np.float32(4.0))


def test_stats_accumulates_over_chunks_and_not_over_transposed_axis():
    g = torch.Generator().manual_seed(2)
    X = torch.randn(40, 6, generator=g).to(torch.float16)
    full = oracle.collect_stats(_u16(X), oracle.F16)
    part = oracle.collect_stats(_u16(X[:25]), oracle.F16)
    part = oracle.collect_stats(_u16(X[25:]), oracle.F16, part)
    np.testing.assert_allclose(part, full, rtol=1e-15)
    # reducing over the wrong axis would give 40 values / other numbers
    assert full.shape == (6,)
    np.testing.assert_allclose(full, (X.double().numpy() ** 2).sum(0), rtol=1e-14)


# ----------------------------------------------------------------------------- Algorithm 1
@pytest.mark.parametrize("d_in", [1, 7, 100, 512, 4096, 11008])
@pytest.mark.parametrize("b", [2.0, 2.2, 2.5, 2.75, 3.0, 3.1, 3.5, 3.999, 4.0])
def test_alloc_budget_and_monotonicity(d_in, b):
    rng = np.random.default_rng(d_in)
    a = np.exp(rng.standard_normal(d_in)).astype(np.float32)
    bits, order = oracle.allocate_bits(a, b)
    assert set(np.unique(bits)) <= {2, 3, 4}
    # I1: the budget is met to within half a channel, exactly when |b-3| d_in is an integer
    if b != 3.0:
        assert abs(bits.mean() - b) <= 0.5 / d_in + 1e-12
        t = abs(b - 3.0) * d_in
        if abs(t - round(t)) < 1e-9:
            assert bits.astype(np.int64).sum() == round(b * d_in)
    else:
        assert bits.astype(np.int64).sum() == 3 * d_in  # symmetric 1 % / 1 %
    # I2: a larger statistic never gets fewer bits
    srt = np.argsort(a, kind="stable")
    assert np.all(np.diff(bits[srt].astype(int)) >= 0)
    # order is the stable ascending argsort
    assert np.array_equal(order, srt.astype(np.int32))
    # one-sided branches never mix 2 and 4 bits
    if b > 3.0:
        assert 2 not in bits
    if b < 3.0:
        assert 4 not in bits


def test_alloc_extremes_and_paper_facts():
    facts = _facts()
    a = np.linspace(1.0, 2.0, 1000).astype(np.float32)
    assert np.all(oracle.allocate_bits(a, 2.0)[0] == 2)
    assert np.all(oracle.allocate_bits(a, 4.0)[0] == 4)
    bits, _ = oracle.allocate_bits(a, 3.0)
    assert (bits == 4).mean() == pytest.approx(facts["frac_4bit_at_b3"], abs=1e-3)
    assert (bits == 2).mean() == pytest.approx(facts["frac_2bit_at_b3"], abs=1e-3)
    # the largest statistics are the ones that get 4 bits, the smallest get 2
    assert np.all(bits[-10:] == 4) and np.all(bits[:10] == 2) and np.all(bits[10:-10] == 3)
    # "2 -> 2.2 bits is a 10 % increase in storage"
    b22 = oracle.allocate_bits(a, 2.2)[0].astype(np.int64).sum()
    b20 = oracle.allocate_bits(a, 2.0)[0].astype(np.int64).sum()
    assert b22 / b20 == pytest.approx(facts["storage_ratio_2p2_over_2"], abs=1e-3)
    with pytest.raises(ValueError):
        oracle.allocate_bits(a, 1.9)
    with pytest.raises(ValueError):
        oracle.allocate_bits(a, 4.1)


def test_alloc_counts_at_the_workload_sizes():
    assert oracle.alloc_counts(4096, 2.2) == (3277, 0)
    assert oracle.alloc_counts(4096, 2.5) == (2048, 0)
    assert oracle.alloc_counts(11008, 3.5) == (0, 5504)
    assert oracle.alloc_counts(512, 3.0) == (5, 5)
    assert oracle.alloc_counts(4096, 3.0) == (41, 41)
    assert oracle.alloc_counts(28672, 2.5) == (14336, 0)


def test_alloc_ties_go_by_channel_id():
    a = np.array([1, 1, 1, 1, 1, 1, 1, 1, 1, 1], np.float32)
    bits, order = oracle.allocate_bits(a, 2.5)
    assert np.array_equal(order, np.arange(10))
    assert np.array_equal(bits, [2] * 5 + [3] * 5)
    bits, _ = oracle.allocate_bits(a, 3.3)
    assert np.array_equal(bits, [3] * 7 + [4] * 3)


@pytest.mark.parametrize("b", [2.2, 2.5, 3.0, 3.4, 3.75])
def test_alloc_literal_mode_matches_library_quantile(b):
    rng = np.random.default_rng(5)
    a = np.exp(rng.standard_normal(2001)).astype(np.float32)
    bits, _ = oracle.allocate_bits(a, b, mode=1)
    ref = np.full(a.shape, 3, np.uint8)
    a64 = a.astype(np.float64)
    if b > 3:
        ref[a64 > np.quantile(a64, 1 - (b - 3))] = 4
    elif b < 3:
        ref[a64 < np.quantile(a64, 3 - b)] = 2
    else:
        ref[a64 < np.quantile(a64, 0.01)] = 2
        ref[a64 > np.quantile(a64, 0.99)] = 4
    assert np.array_equal(bits, ref)
    # the rank form differs from the literal one by a channel or two at most
    rank_bits, _ = oracle.allocate_bits(a, b, mode=0)
    assert np.count_nonzero(rank_bits != bits) <= 2


def test_default_outlier_counts_respect_the_paper_budget():
    facts = _facts()
    for d_in, d_out, na, nq in [(512, 512, 2, 131), (4096, 4096, 18, 8388), (4096, 11008, 18, 22544),
                                (11008, 4096, 49, 22544), (8192, 28672, 36, 117440),
                                (28672, 8192, 129, 117440)]:
        n_act, n_q = oracle.default_counts(d_in, d_out)
        assert (n_act, n_q) == (na, nq)
        assert n_act <= facts["outlier_frac_act"] * d_in
        assert n_q <= facts["outlier_frac_q"] * d_in * d_out
        assert (n_act * d_out + n_q) <= facts["outlier_frac_total"] * d_in * d_out
