"""GPU parity of the calls whose last assignment writes the packed bit streams itself
(cmpq_quantize_layer_packed, cmpq_protect_quantize_pack) against the CPU checker's final fit and packer:
packed words, layout, codes and tables bit for bit, with and without the byte codes materialised."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_13056_b200 import binding as B
from paper_2410_13056_b200 import inputs
from paper_2410_13056_b200.pipeline import LayerQuantizer

import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.fixture(params=["ordered", "all_pairs"])
def assignment(request):
    B.cmpq_set_lloyd_assignment(B.ASSIGN_ALL_PAIRS if request.param == "all_pairs" else B.ASSIGN_ORDERED)
    yield request.param
    B.cmpq_set_lloyd_assignment(B.ASSIGN_ORDERED)


def _case(d_in, d_out, dtype, seed):
    W = inputs.make_weight(d_in, d_out, dtype, seed, device="cuda")
    bits = np.full(d_in, 3, np.uint8)
    bits[: d_in // 3] = 2
    bits[d_in // 3: 2 * d_in // 3] = 4
    bits = bits[np.random.default_rng(seed).permutation(d_in)]
    return W, inputs.as_u16(W), bits


def _packed_buffers(bits, d_in, d_out):
    words = oracle.packed_words(bits, d_out)
    packed = torch.full((words + 8,), -1, dtype=torch.int32, device="cuda")
    row_off = torch.full((d_in + 1,), -1, dtype=torch.int64, device="cuda")
    perm = torch.full((d_in,), -1, dtype=torch.int32, device="cuda")
    seg = torch.full((3,), -1, dtype=torch.int64, device="cuda")
    return words, packed, row_off, perm, seg


def _assert_packed(words, packed, row_off, perm, seg, rcodes, bits):
    p = packed.cpu().numpy().view(np.uint32)
    assert np.all(p[words:] == 0xffffffff), "wrote past the end of the packed words"
    rp, rro, rperm, rseg = oracle.pack(rcodes, bits)
    assert np.array_equal(p[:words], rp)
    assert np.array_equal(row_off.cpu().numpy(), rro) and np.array_equal(perm.cpu().numpy(), rperm)
    assert np.array_equal(seg.cpu().numpy(), rseg)


@pytest.mark.parametrize("dtype", [inputs.F16, inputs.BF16])
@pytest.mark.parametrize("with_codes", [True, False])
@pytest.mark.parametrize("d_in,d_out,T", [(96, 512, 10), (40, 1000, 6), (24, 4096, 8), (12, 11008, 5), (6, 28672, 4),
                                          (50, 37, 12), (64, 16, 9), (9, 1, 3), (23, 31, 3), (23, 33, 3), (7, 8, 2),
                                          (5, 32768, 2), (30, 2056, 4), (30, 2052, 4)])
def test_quantize_layer_packed_matches_checker(dtype, with_codes, d_in, d_out, T, assignment):
    W, Wu, bits = _case(d_in, d_out, dtype, 90 + d_out)
    rng = np.random.default_rng(d_out)
    nnz = min(d_in * d_out // 50, 600)
    lin = np.sort(rng.choice(d_in * d_out, nnz, replace=False))
    rows, cols = (lin // d_out).astype(np.int32), (lin % d_out).astype(np.int32)
    words, packed, row_off, perm, seg = _packed_buffers(bits, d_in, d_out)
    lut = torch.full((d_in, 16), -7.0, dtype=torch.float32, device="cuda")
    codes = torch.full((d_in, d_out), 255, dtype=torch.uint8, device="cuda") if with_codes else None
    call = lambda: B.cmpq_quantize_layer_packed(
        W, G.dev(bits), G.dev(rows) if nnz else None, G.dev(cols) if nnz else None, T, lut, codes, packed[:words],
        row_off, perm, seg, B.workspace(B.OP_QUANTIZE_LAYER_PACKED, d_in, d_out))
    if not with_codes and assignment == "all_pairs":
        with pytest.raises(B.CmpqError) as e:      # that kernel can only produce byte codes
            call()
        assert e.value.status == 2
        return
    call()
    torch.cuda.synchronize()
    rlut, rcodes = oracle.quantize_layer(Wu, dtype, bits, rows, cols, T)
    _assert_packed(words, packed, row_off, perm, seg, rcodes, bits)
    assert np.array_equal(lut.cpu().numpy().view(np.uint32), rlut.view(np.uint32))
    if with_codes:
        assert np.array_equal(codes.cpu().numpy(), rcodes)


def test_quantize_layer_packed_degenerate_channels_and_removed_positions():
    """All-zero, constant and two-valued channels (their centroids are not strictly increasing, so the last
    assignment takes the defining scan), rows with few and with many removed positions, a strided W."""
    d_out = 600
    rows_ = [np.zeros(d_out), np.full(d_out, 0.375), np.where(np.arange(d_out) % 8 == 0, -3.0, 1.0),
             np.linspace(-1, 1, d_out), np.arange(d_out) % 3 - 1.0, np.linspace(-2, 5, d_out) ** 3]
    wide = torch.zeros((len(rows_), d_out + 8), dtype=torch.float16, device="cuda")
    wide[:, :d_out] = torch.tensor(np.stack(rows_), dtype=torch.float16)
    Wt = wide[:, :d_out]                                    # ldw = d_out + 8
    Wu = inputs.as_u16(Wt)
    lin = np.sort(np.concatenate([3 * d_out + np.arange(0, 40), 5 * d_out + np.arange(100, 105), [2 * d_out + 8]]))
    rows, cols = (lin // d_out).astype(np.int32), (lin % d_out).astype(np.int32)
    for c in (2, 3, 4):
        bits = np.full(len(rows_), c, np.uint8)
        words, packed, row_off, perm, seg = _packed_buffers(bits, len(rows_), d_out)
        lut = torch.empty((len(rows_), 16), dtype=torch.float32, device="cuda")
        B.cmpq_quantize_layer_packed(Wt, G.dev(bits), G.dev(rows), G.dev(cols), 7, lut, None, packed[:words], row_off,
                                     perm, seg, B.workspace(B.OP_QUANTIZE_LAYER_PACKED, len(rows_), d_out))
        torch.cuda.synchronize()
        rlut, rcodes = oracle.quantize_layer(Wu, inputs.F16, bits, rows, cols, 7)
        _assert_packed(words, packed, row_off, perm, seg, rcodes, bits)
        assert np.array_equal(lut.cpu().numpy().view(np.uint32), rlut.view(np.uint32))


@pytest.mark.parametrize("dtype", [inputs.F16, inputs.BF16])
@pytest.mark.parametrize("with_codes", [True, False])
@pytest.mark.parametrize("d_in,d_out,n_act,n_q,T", [(64, 512, 2, 40, 8), (33, 4096, 1, 500, 10), (20, 64, 0, 0, 3),
                                                    (6, 1024, 1, 900, 5), (10, 50, 2, 8 * 50, 4), (5, 1, 1, 2, 3),
                                                    (48, 1000, 0, 77, 5)])
def test_protect_quantize_pack_matches_checker(dtype, with_codes, d_in, d_out, n_act, n_q, T):
    W, Wu, bits = _case(d_in, d_out, dtype, 190 + d_in)
    a = np.random.default_rng(d_in).random(d_in).astype(np.float32)
    nnz = n_act * d_out + n_q
    r = torch.full((max(nnz, 1),), -1, dtype=torch.int32, device="cuda")
    c = torch.full((max(nnz, 1),), -1, dtype=torch.int32, device="cuda")
    v = torch.zeros(max(nnz, 1), dtype=torch.int16, device="cuda")
    lut = torch.full((d_in, 16), -7.0, dtype=torch.float32, device="cuda")
    codes = torch.full((d_in, d_out), 255, dtype=torch.uint8, device="cuda") if with_codes else None
    words, packed, row_off, perm, seg = _packed_buffers(bits, d_in, d_out)
    B.cmpq_protect_quantize_pack(W, G.dev(a), G.dev(bits), n_act, n_q, T, r[:nnz], c[:nnz], v[:nnz], lut, codes,
                                 packed[:words], row_off, perm, seg,
                                 B.workspace(B.OP_PROTECT_QUANTIZE_PACK, d_in, d_out))
    torch.cuda.synchronize()
    rr, rc, rv = oracle.extract_outliers(Wu, dtype, a, bits, n_act, n_q, T)
    assert np.array_equal(r[:nnz].cpu().numpy(), rr) and np.array_equal(c[:nnz].cpu().numpy(), rc)
    assert np.array_equal(v[:nnz].cpu().numpy().view(np.uint16), rv)
    rlut, rcodes = oracle.quantize_layer(Wu, dtype, bits, rr, rc, T)
    _assert_packed(words, packed, row_off, perm, seg, rcodes, bits)
    assert np.array_equal(lut.cpu().numpy().view(np.uint32), rlut.view(np.uint32))
    if with_codes:
        assert np.array_equal(codes.cpu().numpy(), rcodes)


def test_pass_without_byte_codes_equals_the_pass_with_them():
    d_in, d_out, n, T = 256, 1536, 2048, 12
    W = inputs.make_weight(d_in, d_out, inputs.BF16, 31, device="cuda")
    X = inputs.make_activations(n, d_in, inputs.BF16, 31, device="cuda")
    full = G.result_arrays(LayerQuantizer(d_in, d_out).run(X, W, 2.5, T))
    q = LayerQuantizer(d_in, d_out, keep_codes=False)
    r = q.run_graphed(X, W, 2.5, T)
    assert r.codes is None
    torch.cuda.synchronize()
    for k in ("bits", "rows", "cols", "lut", "row_off", "perm", "seg_rows"):
        assert np.array_equal(getattr(r, k).cpu().numpy(), full[k]), k
    assert np.array_equal(r.packed.cpu().numpy().view(np.uint32), full["packed"])
    codes = oracle.unpack(full["packed"], full["row_off"], full["perm"], full["bits"], d_out)
    assert np.array_equal(codes, full["codes"])
