"""GPU parity of the inference product (Section 6 of the paper) and of the outlier list by column.

Inputs are random already-quantized layers from the seeded generator, packed by the CPU checker; the
library reads those packed segments and its result is compared column by column with the checker's
fp64 sum.  Tolerance: every product x_i * lut_i[k] is rounded once to fp32 and a column is summed in
fp32 through at most ~100 sequential additions per path (<= 64 channels per warp, 8 warps, chunks / 8
partials per finishing warp, 8 warps, the outlier term), so
    |y_gpu - y| <= 100 * 2^-24 * sum_i |x_i w_ij| < 1e-5 * yabs;  the tests allow 2e-5 * yabs."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import dev
from paper_2410_13056_b200 import binding as B
from paper_2410_13056_b200 import inputs
from paper_2410_13056_b200.pipeline import LayerQuantizer, QuantizedLinear

pytestmark = pytest.mark.gpu
TOL = 2e-5


def _gpu_by_column(q, d_out):
    nnz = q["rows"].size
    col_ptr = torch.full((d_out + 1,), -1, dtype=torch.int64, device="cuda")
    c_rows = torch.full((nnz + 4,), -1, dtype=torch.int32, device="cuda")
    c_vals = torch.full((nnz + 4,), -1, dtype=torch.int16, device="cuda")
    rows, cols, vals = (dev(q["rows"]), dev(q["cols"]), dev(q["vals"].view(np.int16))) if nnz else (None,) * 3
    B.cmpq_outliers_by_column(rows, cols, vals, d_out, col_ptr, c_rows, c_vals,
                              B.workspace(B.OP_OUTLIERS_BY_COLUMN, 1, d_out))
    torch.cuda.synchronize()
    assert torch.all(c_rows[nnz:] == -1) and torch.all(c_vals[nnz:] == -1)
    return col_ptr, c_rows[:nnz], c_vals[:nnz]


def _gpu_matvec(q, dtype, want16=True, with_outliers=True):
    d_in, d_out = q["codes"].shape
    packed, row_off, perm, seg = oracle.pack(q["codes"], q["bits"])
    col_ptr = c_rows = c_vals = None
    if with_outliers and q["rows"].size:
        col_ptr, c_rows, c_vals = _gpu_by_column(q, d_out)
    x = dev(q["x"].view(np.int16)).view(inputs.torch_dtype(dtype))
    y = torch.full((d_out + 3,), 7.0, dtype=torch.float32, device="cuda")
    y16 = torch.full((d_out + 3,), 7.0, dtype=inputs.torch_dtype(dtype), device="cuda") if want16 else None
    pk = torch.zeros(packed.size + 8, dtype=torch.int32, device="cuda")   # 16-byte aligned base
    pk[:packed.size] = dev(packed.view(np.int32))
    B.cmpq_matvec(pk, dev(row_off), dev(perm), dev(seg), dev(q["lut"]), x, col_ptr, c_rows, c_vals,
                  y[:d_out], None if y16 is None else y16[:d_out], B.workspace(B.OP_MATVEC, d_in, d_out))
    torch.cuda.synchronize()
    assert torch.all(y[d_out:] == 7.0)
    return y[:d_out].cpu().numpy(), (None if y16 is None else y16[:d_out])


def _check(q, dtype, y, y16=None, with_outliers=True):
    none = (np.zeros(0, np.int32), np.zeros(0, np.int32), np.zeros(0, np.uint16))
    o = (q["rows"], q["cols"], q["vals"]) if with_outliers else none
    ref, yabs = oracle.matvec(q["x"], dtype, q["lut"], q["codes"], *o)
    assert np.all(np.abs(y.astype(np.float64) - ref) <= TOL * yabs + 1e-37), \
        float(np.max(np.abs(y - ref) / (yabs + 1e-300)))
    if y16 is not None:
        # the 16-bit output is the fp32 output rounded to nearest even
        assert torch.equal(y16.cpu(), torch.from_numpy(y).to(y16.dtype))
    return ref, yabs


@pytest.mark.parametrize("dtype", [inputs.F16, inputs.BF16])
@pytest.mark.parametrize("shape,counts,n_act,n_q", [
    ((33, 16), (11, 11, 11), 1, 5),            # fewer columns than one group of 32
    ((40, 72), (40, 0, 0), 0, 9),              # one width only, ragged last group
    ((72, 40), (0, 72, 0), 2, 0),
    ((130, 1000), (0, 0, 130), 0, 0),          # no outliers at all
    ((257, 1030), (100, 57, 100), 3, 300),     # two column tiles, ragged tail, odd word counts
    ((700, 2080), (3, 690, 7), 4, 900),        # several chunks per segment, short segments
    ((1200, 4096), (600, 200, 400), 5, 2400),
    ((70, 32768), (20, 30, 20), 1, 500),       # the widest layer the library takes
])
def test_matvec_against_the_checker(dtype, shape, counts, n_act, n_q):
    q = inputs.make_quantized_layer(shape[0], shape[1], counts, dtype, 17 + shape[0], n_act, n_q)
    y, y16 = _gpu_matvec(q, dtype)
    _check(q, dtype, y, y16)
    y2, _ = _gpu_matvec(q, dtype, want16=False)
    assert np.array_equal(y, y2)               # same bytes on a second call
    y3, _ = _gpu_matvec(q, dtype, with_outliers=False)
    _check(q, dtype, y3, with_outliers=False)


@pytest.mark.parametrize("shape,n_act,n_q", [((64, 48), 2, 40), ((300, 1030), 3, 999), ((96, 32768), 1, 5000),
                                             ((3000, 16), 2900, 100)])
def test_outliers_by_column_bit_exact(shape, n_act, n_q):
    d_in, d_out = shape
    q = inputs.make_quantized_layer(d_in, d_out, (d_in, 0, 0), inputs.BF16, 5, n_act, n_q)
    col_ptr, c_rows, c_vals = _gpu_by_column(q, d_out)
    ref = oracle.outliers_by_column(q["rows"], q["cols"], q["vals"], d_out)
    assert np.array_equal(col_ptr.cpu().numpy(), ref[0])
    assert np.array_equal(c_rows.cpu().numpy(), ref[1])
    assert np.array_equal(c_vals.cpu().numpy().view(np.uint16), ref[2])
    empty = dict(q, rows=np.zeros(0, np.int32), cols=np.zeros(0, np.int32), vals=np.zeros(0, np.uint16))
    col_ptr0, _, _ = _gpu_by_column(empty, d_out)
    assert np.array_equal(col_ptr0.cpu().numpy(), np.zeros(d_out + 1, np.int64))


@pytest.mark.parametrize("shape,budget_counts", [((4096, 4096), (41, 4014, 41)),        # attention, 3.0 bits
                                                 ((4096, 11008), (2048, 2048, 0)),     # MLP up, 2.5 bits
                                                 ((11008, 4096), (0, 5504, 5504))])    # MLP down, 3.5 bits
def test_matvec_llama_shapes(shape, budget_counts):
    d_in, d_out = shape
    n_act, n_q = B.cmpq_default_counts(d_in, d_out)
    q = inputs.make_quantized_layer(d_in, d_out, budget_counts, inputs.BF16, 23, n_act, n_q)
    y, y16 = _gpu_matvec(q, inputs.BF16)
    _check(q, inputs.BF16, y, y16)


def test_matvec_after_the_quantization_pass():
    """The product reads what the pass wrote: quantize a layer on the device, multiply a token, and
    compare with the checker's product evaluated from the SAME look-up tables, codes and outliers."""
    d_in, d_out, n, T = 384, 1536, 1024, 8
    W = inputs.make_weight(d_in, d_out, inputs.BF16, 41, device="cuda")
    X = inputs.make_activations(n, d_in, inputs.BF16, 41, device="cuda")
    quant = LayerQuantizer(d_in, d_out)
    r = quant.run(X, W, 2.75, T)
    layer = QuantizedLinear.from_result(r)
    y16 = torch.empty(d_out, dtype=torch.bfloat16, device="cuda")
    y = layer.matvec(X[3], y16).cpu().numpy()
    ref, yabs = oracle.matvec(inputs.as_u16(X[3]), inputs.BF16, r.lut.cpu().numpy(), r.codes.cpu().numpy(),
                              r.rows.cpu().numpy(), r.cols.cpu().numpy(), r.vals.cpu().numpy().view(np.uint16))
    assert np.all(np.abs(y - ref) <= TOL * yabs)
    # and it approximates the unquantized product: the error is the token's share of ||X (W - What)||
    exact = X[3].double().cpu().numpy() @ W.double().cpu().numpy()
    assert np.linalg.norm(y - exact) < 0.2 * np.linalg.norm(exact)


def test_matvec_argument_checks():
    q = inputs.make_quantized_layer(64, 64, (64, 0, 0), inputs.BF16, 1)
    packed, row_off, perm, seg = oracle.pack(q["codes"], q["bits"])
    x = dev(q["x"].view(np.int16)).view(torch.bfloat16)
    y = torch.zeros(64, dtype=torch.float32, device="cuda")
    args = [dev(packed.view(np.int32)), dev(row_off), dev(perm), dev(seg), dev(q["lut"]), x, None, None, None, y, None]
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.CmpqError) as e:
        B.cmpq_matvec(*args, small[:0])
    assert e.value.status == 3
    with pytest.raises(B.CmpqError) as e:   # a column index without its lists
        B.cmpq_matvec(*(args[:6] + [torch.zeros(65, dtype=torch.int64, device="cuda"), None, None, y, None]),
                      B.workspace(B.OP_MATVEC, 64, 64))
    assert e.value.status == 1
    torch.cuda.synchronize()
    assert torch.all(y == 0)
