"""GPU parity of the stored table formats (Section 5.1 of the paper: FP16 tables, 4-bit variant) and of
the inference product reading FP16 tables.  Conversions are bit-exact; the product keeps the tolerance
of the other inference-product tests."""
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


def _tables(d_in, seed):
    rng = np.random.default_rng(seed)
    bits = rng.integers(2, 5, d_in).astype(np.uint8)
    lut = np.sort(rng.normal(0, 0.02, (d_in, 16)) * 10.0 ** rng.uniform(-3, 2, (d_in, 1)), axis=1).astype(np.float32)
    lut[np.arange(16)[None, :] >= (1 << bits.astype(np.int64))[:, None]] = 0.0
    lut[3, : 1 << int(bits[3])] = -0.375                      # constant channel: zero step
    lut[5, 0] = -70000.0                                      # beyond the binary16 range
    lut[6, :4] = [0.0, 2.0 ** -25, 2.0 ** -24, 3 * 2.0 ** -25]  # binary16 subnormals and ties
    lut[7, : 1 << int(bits[7])] = rng.permutation(lut[7, : 1 << int(bits[7])])   # unsorted centroids
    return bits, lut


def _store(lut, bits, fmt):
    d_in = lut.shape[0]
    n = B.cmpq_lut_bytes(fmt, d_in)
    out = torch.full((n + 8,), 0x5a, dtype=torch.uint8, device="cuda")
    B.cmpq_store_lut(dev(lut), dev(bits), fmt, out)
    torch.cuda.synchronize()
    assert torch.all(out[n:] == 0x5a)
    return out[:n]


@pytest.mark.parametrize("d_in", [9, 257, 4096])
def test_store_and_load_are_bit_exact(d_in):
    bits, lut = _tables(d_in, d_in)
    assert B.cmpq_lut_bytes(B.LUT_F16, d_in) == d_in * 32 and B.cmpq_lut_bytes(B.LUT_U4, d_in) == d_in * 12
    s16 = _store(lut, bits, B.LUT_F16)
    with np.errstate(over="ignore"):
        ref16 = oracle.lut_to_f16(lut, bits)
    assert np.array_equal(s16.cpu().numpy().view(np.uint16).reshape(d_in, 16), ref16)
    su4 = _store(lut, bits, B.LUT_U4)
    refu4 = oracle.lut_to_u4(lut, bits)
    keep = np.ones(d_in, bool)
    keep[5] = False                                            # an infinite grid end has no defined codes
    assert np.array_equal(su4.cpu().numpy().reshape(d_in, 12)[keep], refu4[keep])
    back = torch.full((d_in, 16), 9.0, dtype=torch.float32, device="cuda")
    B.cmpq_load_lut(s16, B.LUT_F16, dev(bits), back)
    torch.cuda.synchronize()
    assert np.array_equal(back.cpu().numpy().view(np.uint32), oracle.lut_from_f16(ref16).view(np.uint32))
    B.cmpq_load_lut(su4, B.LUT_U4, dev(bits), back)
    torch.cuda.synchronize()
    assert np.array_equal(back.cpu().numpy()[keep].view(np.uint32), oracle.lut_from_u4(refu4, bits)[keep].view(np.uint32))


def test_stored_tables_of_a_quantized_layer_and_their_overhead():
    """A layer quantized on the device: its tables in both stored formats equal the checker's conversion
    of the checker's tables, the 4-bit tables reproduce every centroid within half a grid step, and the
    overhead figures are the paper's."""
    d_in, d_out, n, T = 256, 4096, 1024, 10
    W = inputs.make_weight(d_in, d_out, inputs.BF16, 71, device="cuda")
    X = inputs.make_activations(n, d_in, inputs.BF16, 71, device="cuda")
    q = LayerQuantizer(d_in, d_out)
    r = q.run(X, W, 3.0, T)
    bits = r.bits.cpu()
    s16 = torch.empty(d_in * 16, dtype=torch.int16, device="cuda")
    su4 = torch.empty(d_in * 12, dtype=torch.uint8, device="cuda")
    B.cmpq_store_lut(r.lut, r.bits, B.LUT_F16, s16)
    B.cmpq_store_lut(r.lut, r.bits, B.LUT_U4, su4)
    lut = r.lut.cpu().numpy()
    assert np.array_equal(s16.cpu().numpy().view(np.uint16).reshape(d_in, 16), oracle.lut_to_f16(lut, bits.numpy()))
    assert np.array_equal(su4.cpu().numpy().reshape(d_in, 12), oracle.lut_to_u4(lut, bits.numpy()))
    dec = oracle.lut_from_u4(su4.cpu().numpy().reshape(d_in, 12), bits.numpy())
    K = (1 << bits.numpy().astype(np.int64))
    for i in range(d_in):
        c = lut[i, :K[i]]
        assert np.all(np.abs(dec[i, :K[i]] - c) <= (c.max() - c.min()) / 30 + 2e-3 * np.abs(c).max() + 1e-12)
    f16 = B.cmpq_table_bits_per_weight(bits, d_out, B.LUT_F16)
    u4 = B.cmpq_table_bits_per_weight(bits, d_out, B.LUT_U4)
    assert f16 == oracle.metadata_bits_per_weight(bits.numpy(), d_out, 4, 16) and 0.03 < f16 < 0.034
    assert u4 == oracle.metadata_bits_per_weight(bits.numpy(), d_out, 4, 4) and u4 < 0.01
    assert B.cmpq_table_bits_per_weight(bits, d_out, B.LUT_U4, True) == pytest.approx(u4 + 32 / d_out)


@pytest.mark.parametrize("dtype", [inputs.F16, inputs.BF16])
@pytest.mark.parametrize("shape,counts,n_act,n_q", [((257, 1030), (100, 57, 100), 3, 300),
                                                    ((1200, 4096), (600, 200, 400), 5, 2400)])
def test_matvec_reading_fp16_tables(dtype, shape, counts, n_act, n_q):
    q = inputs.make_quantized_layer(shape[0], shape[1], counts, dtype, 23 + shape[0], n_act, n_q)
    d_in, d_out = shape
    lut16 = oracle.lut_to_f16(q["lut"], q["bits"])
    lut_rounded = oracle.lut_from_f16(lut16)
    packed, row_off, perm, seg = oracle.pack(q["codes"], q["bits"])
    layer = QuantizedLinear(dev(packed.view(np.int32)), dev(row_off), dev(perm), dev(seg), dev(lut_rounded),
                            dev(q["rows"]), dev(q["cols"]), dev(q["vals"].view(np.int16)), d_out)
    x = dev(q["x"].view(np.int16)).view(inputs.torch_dtype(dtype))
    y32 = layer.matvec(x).clone()                               # fp32 tables holding the rounded values
    y = torch.full((d_out,), 7.0, dtype=torch.float32, device="cuda")
    B.cmpq_matvec_f16lut(layer.packed, layer.row_off, layer.perm, layer.seg_rows, dev(lut16.view(np.int16)), x,
                         layer.col_ptr, layer.c_rows, layer.c_vals, y, None, layer.ws)
    torch.cuda.synchronize()
    assert torch.equal(y, y32)                                  # widening is exact: the same bytes
    ref, yabs = oracle.matvec(q["x"], dtype, lut_rounded, q["codes"], q["rows"], q["cols"], q["vals"])
    assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - ref) <= TOL * yabs + 1e-37)
