"""GPU parity of the sensitivity-weighted channel K-means (cmpq_quantize_layer with sens) against the
checker.  The weighted sums s_i x_i are not exact in fp64, so the two sides may round a centroid
differently in the last place: centroids are compared at 1e-4 relative (floor 1e-4 of the channel's largest
magnitude), codes must be identical wherever the two sides' centroids are bit-equal and must in any case be
a nearest centroid (first minimum) under the library's own centroids.  With equal sensitivities the
weighted kernel must reproduce the unweighted fit bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import gpu_util as G
from paper_2410_13056_b200 import inputs

pytestmark = pytest.mark.gpu


def _bits(d_in, seed):
    return np.random.default_rng(seed).integers(2, 5, d_in).astype(np.uint8)


def _outliers(d_in, d_out, n, seed):
    g = np.random.default_rng(seed)
    lin = np.sort(g.choice(d_in * d_out, size=n, replace=False))
    return (lin // d_out).astype(np.int32), (lin % d_out).astype(np.int32)


def _first_min_codes(x, lut, K):
    d = np.abs(x[:, None].astype(np.float32) - lut[None, :K].astype(np.float32))
    return np.argmin(d, axis=1).astype(np.uint8)      # argmin returns the first minimum


@pytest.mark.parametrize("dtype", [inputs.F16, inputs.BF16])
@pytest.mark.parametrize("shape,T,nnz", [((24, 512), 10, 0), ((40, 1000), 20, 300), ((7, 4096), 20, 50), ((3, 16), 5, 4),
                                         ((5, 32768), 8, 100)])   # the widest channel the library takes
def test_weighted_fit_against_the_checker(dtype, shape, T, nnz):
    d_in, d_out = shape
    W = inputs.make_weight(d_in, d_out, dtype, 100 + d_out, device="cuda")
    bits = _bits(d_in, d_out)
    rows, cols = _outliers(d_in, d_out, nnz, 3)
    g = torch.Generator(device="cuda")
    g.manual_seed(d_out)
    sens = (torch.rand((d_in, d_out), device="cuda", generator=g) ** 2 * 4 + 0.01).float()
    lut, codes, _, sweeps = G.gpu_quantize(W, bits, rows, cols, T, sens=sens)
    ref_lut, ref_codes = oracle.quantize_layer(inputs.as_u16(W), dtype, bits, rows, cols, T,
                                               sens=sens.double().cpu().numpy())
    Wf = W.float().cpu().numpy().copy()
    Wf[rows, cols] = 0.0
    Wf = Wf + np.float32(0.0)
    for i in range(d_in):
        K = 1 << int(bits[i])
        floor = 1e-4 * max(np.abs(Wf[i]).max(), 1e-30)
        assert np.all(np.abs(lut[i] - ref_lut[i]) <= 1e-4 * np.abs(ref_lut[i]) + floor), i
        assert np.all(lut[i, K:] == 0)
        assert np.array_equal(codes[i], _first_min_codes(Wf[i], lut[i], K)), i          # valid under its own centroids
        if np.array_equal(lut[i].view(np.uint32), ref_lut[i].view(np.uint32)):
            assert np.array_equal(codes[i], ref_codes[i]), i
    same = sum(np.array_equal(lut[i].view(np.uint32), ref_lut[i].view(np.uint32)) for i in range(d_in))
    assert same >= 0.8 * d_in                                                          # rounding differences are rare
    assert sweeps > 0


@pytest.mark.parametrize("dtype", [inputs.F16, inputs.BF16])
def test_equal_sensitivities_reproduce_the_unweighted_fit(dtype):
    d_in, d_out, T = 48, 1536, 15
    W = inputs.make_weight(d_in, d_out, dtype, 7, device="cuda")
    bits = _bits(d_in, 1)
    rows, cols = _outliers(d_in, d_out, 200, 5)
    base_lut, base_codes, inexact, _ = G.gpu_quantize(W, bits, rows, cols, T)
    assert inexact == 0
    for value in (1.0, 0.25):     # powers of two: s*x and the sums stay exact, so the order cannot matter
        sens = torch.full((d_in, d_out), value, dtype=torch.float32, device="cuda")
        lut, codes, _, _ = G.gpu_quantize(W, bits, rows, cols, T, sens=sens)
        assert np.array_equal(lut.view(np.uint32), base_lut.view(np.uint32))
        assert np.array_equal(codes, base_codes)
    # and a second run gives the same bytes
    sens = torch.rand((d_in, d_out), device="cuda") + 0.5
    a = G.gpu_quantize(W, bits, rows, cols, T, sens=sens)
    b = G.gpu_quantize(W, bits, rows, cols, T, sens=sens)
    assert np.array_equal(a[0].view(np.uint32), b[0].view(np.uint32)) and np.array_equal(a[1], b[1])


def test_zero_sensitivity_cluster_keeps_its_centroid():
    # sensitivities 0 on every weight of a channel: no centroid may move from the start
    d_in, d_out = 2, 256
    W = inputs.make_weight(d_in, d_out, inputs.BF16, 9, device="cuda")
    bits = np.array([3, 2], np.uint8)
    none = np.zeros(0, np.int32)
    sens = torch.zeros((d_in, d_out), dtype=torch.float32, device="cuda")
    lut, codes, _, _ = G.gpu_quantize(W, bits, none, none, 6, sens=sens)
    start, start_codes, _, _ = G.gpu_quantize(W, bits, none, none, 0)
    assert np.array_equal(lut.view(np.uint32), start.view(np.uint32)) and np.array_equal(codes, start_codes)


@pytest.mark.parametrize("dtype,shape", [(inputs.BF16, (64, 4096)), (inputs.F16, (12, 4096)), (inputs.F16, (3, 24576))])
def test_table_formulation_agrees_with_the_all_weights_kernel(dtype, shape):
    """The default weighted fit works on the value tables (sums of sensitivities per distinct value); the kernel
    that scans every weight stays selectable through the all-pairs switch.  Same method, different orders of
    summation: centroids agree to rounding, codes wherever the centroids are bit-equal.  bf16 channels of 4096
    weights fit the small table capacity, fp16 ones need the large one, and a 24576-wide fp16 channel has more
    distinct values than shared memory holds and is handed to the all-weights kernel."""
    from paper_2410_13056_b200 import binding as B
    d_in, d_out = shape
    W = inputs.make_weight(d_in, d_out, dtype, 31 + d_out, device="cuda")
    bits = _bits(d_in, 5)
    rows, cols = _outliers(d_in, d_out, 40, 11)
    g = torch.Generator(device="cuda")
    g.manual_seed(17)
    sens = (torch.rand((d_in, d_out), device="cuda", generator=g) * 3 + 0.05).float()
    lut_t, codes_t, _, _ = G.gpu_quantize(W, bits, rows, cols, 12, sens=sens)
    B.cmpq_set_lloyd_assignment(B.ASSIGN_ALL_PAIRS)
    try:
        lut_a, codes_a, _, _ = G.gpu_quantize(W, bits, rows, cols, 12, sens=sens)
    finally:
        B.cmpq_set_lloyd_assignment(B.ASSIGN_ORDERED)
    scale = np.abs(lut_a).max(axis=1, keepdims=True)
    assert np.all(np.abs(lut_t - lut_a) <= 1e-5 * scale)
    equal = [i for i in range(d_in) if np.array_equal(lut_t[i].view(np.uint32), lut_a[i].view(np.uint32))]
    assert len(equal) >= 0.8 * d_in
    for i in equal:
        assert np.array_equal(codes_t[i], codes_a[i]), i
    # and the run is reproducible byte for byte
    lut_2, codes_2, _, _ = G.gpu_quantize(W, bits, rows, cols, 12, sens=sens)
    assert np.array_equal(lut_2.view(np.uint32), lut_t.view(np.uint32)) and np.array_equal(codes_2, codes_t)
