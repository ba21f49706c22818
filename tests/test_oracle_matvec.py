"""Pins for the oracle's inference product (Section 6: per-precision sub-matrix products plus the
outlier product, accumulated) and for the outlier list regrouped by column.  CPU only."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_13056_b200 import inputs


def _quantized(d_in=40, d_out=72, dtype=inputs.BF16, seed=11, budget=3.0, n_act=2, n_q=25, T=5):
    W = inputs.make_weight(d_in, d_out, dtype, seed)
    X = inputs.make_activations(64, d_in, dtype, seed, n_outlier_channels=3)
    Xu, Wu = inputs.as_u16(X), inputs.as_u16(W)
    out = oracle.layer_pass(Xu, Wu, dtype, budget, n_act, n_q, T)
    return X, W, Xu, Wu, out


def _dense_what(out, W_like, dtype, parts=False):
    """What = lut[code] + O as a float64 matrix, built with numpy indexing only."""
    d_in, d_out = out["codes"].shape
    What = np.take_along_axis(out["lut"].astype(np.float64), out["codes"].astype(np.int64), axis=1)
    O = np.zeros((d_in, d_out))
    vals = torch.from_numpy(out["vals"].view(np.int16)).view(inputs.torch_dtype(dtype)).double().numpy()
    O[out["rows"], out["cols"]] = vals
    return (What, O) if parts else What + O


@pytest.mark.parametrize("dtype", [inputs.F16, inputs.BF16])
@pytest.mark.parametrize("shape", [(40, 72), (72, 40), (33, 16)])
def test_matvec_against_dense_float64_product(dtype, shape):
    X, W, Xu, Wu, out = _quantized(shape[0], shape[1], dtype)
    What = _dense_what(out, W, dtype)
    for t in (0, 5):
        y, yabs = oracle.matvec(Xu[t], dtype, out["lut"], out["codes"], out["rows"], out["cols"], out["vals"])
        x = X[t].double().numpy()
        ref = x @ What                                   # library routine, non-square: catches a transpose
        assert np.allclose(y, ref, rtol=0, atol=1e-12 * np.abs(x).max() * np.abs(What).max() * shape[0])
        Q, O = _dense_what(out, W, dtype, parts=True)
        assert np.allclose(yabs, np.abs(x) @ (np.abs(Q) + np.abs(O)), rtol=1e-12, atol=0)
        assert np.all(yabs + 1e-300 >= np.abs(y))


def test_unit_input_reads_one_row_of_the_reconstruction():
    dtype = inputs.BF16
    X, W, Xu, Wu, out = _quantized(dtype=dtype)
    What = _dense_what(out, W, dtype)
    d_in = Wu.shape[0]
    one = inputs.as_u16(torch.ones(1, dtype=inputs.torch_dtype(dtype)))[0]
    for i in (0, 7, d_in - 1, int(out["rows"][0])):
        x = np.zeros(d_in, np.uint16)
        x[i] = one
        y, _ = oracle.matvec(x, dtype, out["lut"], out["codes"], out["rows"], out["cols"], out["vals"])
        assert np.array_equal(y, What[i])                # exact: a single term per column (plus its outlier)


def test_exactly_representable_layer_gives_the_unquantized_product():
    # every channel holds at most 2^c distinct values and T >= 3: the fit is exact (zero error), so the
    # quantized product equals x W evaluated in fp64 term by term
    dtype = inputs.F16
    g = np.random.default_rng(5)
    d_in, d_out = 24, 48
    levels = np.array([-0.5, -0.125, 0.25, 1.0])
    # equal counts per level, shuffled: the evenly spaced starting order statistics hit all four levels
    Wf = np.stack([g.permutation(np.repeat(levels, d_out // 4)) for _ in range(d_in)])
    W = torch.from_numpy(Wf).to(torch.float16)
    X = torch.from_numpy(g.integers(-8, 9, size=(4, d_in)).astype(np.float64)).to(torch.float16)
    Wu, Xu = inputs.as_u16(W), inputs.as_u16(X)
    out = oracle.layer_pass(Xu, Wu, dtype, 2.0, 0, 0, 6)
    assert oracle.recon_error(Xu, Wu, dtype, out["lut"], out["codes"], out["rows"], out["cols"], out["vals"]) == 0.0
    y, _ = oracle.matvec(Xu[1], dtype, out["lut"], out["codes"], out["rows"], out["cols"], out["vals"])
    assert np.array_equal(y, X[1].double().numpy() @ Wf)  # small integers times dyadic levels: exact


def test_matvec_agrees_with_the_reconstruction_error_of_the_layer():
    # E = ||X (W - What)||_F over the tokens equals the norm of (x W - matvec(x)) collected token by token
    dtype = inputs.BF16
    X, W, Xu, Wu, out = _quantized(dtype=dtype)
    E = oracle.recon_error(Xu, Wu, dtype, out["lut"], out["codes"], out["rows"], out["cols"], out["vals"])
    Wd = W.double().numpy()
    total = 0.0
    for t in range(Xu.shape[0]):
        y, _ = oracle.matvec(Xu[t], dtype, out["lut"], out["codes"], out["rows"], out["cols"], out["vals"])
        total += np.sum((X[t].double().numpy() @ Wd - y) ** 2)
    assert np.isclose(np.sqrt(total), E, rtol=1e-9)


def test_outliers_alone_and_codes_alone_add_up():
    dtype = inputs.BF16
    X, W, Xu, Wu, out = _quantized(dtype=dtype)
    none = (np.zeros(0, np.int32), np.zeros(0, np.int32), np.zeros(0, np.uint16))
    y_all, _ = oracle.matvec(Xu[2], dtype, out["lut"], out["codes"], out["rows"], out["cols"], out["vals"])
    y_dense, _ = oracle.matvec(Xu[2], dtype, out["lut"], out["codes"], *none)
    y_sparse, _ = oracle.matvec(Xu[2], dtype, np.zeros_like(out["lut"]), out["codes"], out["rows"], out["cols"],
                                out["vals"])
    # brute force over the list, in python
    x = X[2].double().numpy()
    vals = torch.from_numpy(out["vals"].view(np.int16)).view(torch.bfloat16).double().numpy()
    brute = np.zeros(Wu.shape[1])
    for r, c, v in zip(out["rows"], out["cols"], vals):
        brute[c] += x[r] * v
    assert np.allclose(y_sparse, brute, rtol=1e-13, atol=1e-13)
    assert np.allclose(y_all, y_dense + y_sparse, rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("d_out", [16, 72])
def test_outliers_by_column_is_the_sort_by_column_then_row(d_out):
    dtype = inputs.BF16
    X, W, Xu, Wu, out = _quantized(40, d_out, dtype, n_act=2, n_q=19)
    col_ptr, c_rows, c_vals = oracle.outliers_by_column(out["rows"], out["cols"], out["vals"], d_out)
    nnz = out["rows"].shape[0]
    assert col_ptr[0] == 0 and col_ptr[-1] == nnz and np.all(np.diff(col_ptr) >= 0)
    order = np.lexsort((out["rows"], out["cols"]))      # by column, then row
    assert np.array_equal(c_rows, out["rows"][order])
    assert np.array_equal(c_vals, out["vals"][order])
    assert np.array_equal(np.diff(col_ptr), np.bincount(out["cols"], minlength=d_out))
    empty = oracle.outliers_by_column(np.zeros(0, np.int32), np.zeros(0, np.int32), np.zeros(0, np.uint16), d_out)
    assert np.array_equal(empty[0], np.zeros(d_out + 1, np.int64)) and empty[1].size == 0
