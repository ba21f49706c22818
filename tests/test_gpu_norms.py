"""GPU parity of the l1 and l_inf activation statistics (the paper's norm-ablation criteria) against the
checker: sums within 1e-5 relative (fp32 partial sums of at most 32 magnitudes, fp64 above, as for the
default l2 statistic), the maximum bit for bit; then Algorithm 1 on that criterion, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import gpu_allocate
from paper_2410_13056_b200 import binding as B
from paper_2410_13056_b200 import inputs

pytestmark = pytest.mark.gpu


def _gpu_norm(X, norm, chunks=1):
    n, d_in = X.shape
    acc = torch.zeros(d_in, dtype=torch.float64, device="cuda")
    a = torch.empty(d_in, dtype=torch.float32, device="cuda")
    ws = B.workspace(B.OP_COLLECT_STATS, d_in)
    edges = np.linspace(0, n, chunks + 1).astype(int)
    for lo, hi in zip(edges[:-1], edges[1:]):
        B.cmpq_collect_stats_norm(X[lo:hi], norm, acc, ws)
    B.cmpq_finalize_stats_norm(acc, norm, a)
    torch.cuda.synchronize()
    return acc.cpu().numpy(), a.cpu().numpy()


@pytest.mark.parametrize("dtype", [inputs.F16, inputs.BF16])
@pytest.mark.parametrize("shape,chunks", [((512, 512), 1), ((1000, 100), 3), ((4099, 1032), 2), ((37, 4096), 1),
                                          ((20000, 264), 5)])
def test_norm_statistics_against_the_checker(dtype, shape, chunks):
    X = inputs.make_activations(shape[0], shape[1], dtype, 9 + shape[1], device="cuda")
    Xu = inputs.as_u16(X)
    for norm in (B.NORM_L1, B.NORM_LINF, B.NORM_L2):
        acc, a = _gpu_norm(X, norm, chunks)
        ref = oracle.collect_stats_norm(Xu, dtype, norm)
        ref_a = oracle.finalize_stats_norm(ref, norm)
        if norm == B.NORM_LINF:
            assert np.array_equal(acc, ref) and np.array_equal(a, ref_a)
        else:
            np.testing.assert_allclose(acc, ref, rtol=1e-5)
            np.testing.assert_allclose(a, ref_a, rtol=1e-5)
    # the l2 variant is the default statistic, bit for bit
    sumsq = torch.zeros(shape[1], dtype=torch.float64, device="cuda")
    B.cmpq_collect_stats(X, sumsq, B.workspace(B.OP_COLLECT_STATS, shape[1]))
    assert np.array_equal(sumsq.cpu().numpy(), _gpu_norm(X, B.NORM_L2, 1)[0])


def test_unaligned_rows_take_the_scalar_path():
    X = inputs.make_activations(300, 1001, inputs.BF16, 5, device="cuda")[:, 1:998]   # odd width, odd offset
    Xu = inputs.as_u16(X)
    for norm in (B.NORM_L1, B.NORM_LINF):
        acc, _ = _gpu_norm(X, norm)
        ref = oracle.collect_stats_norm(Xu, inputs.BF16, norm)
        if norm == B.NORM_LINF:
            assert np.array_equal(acc, ref)
        else:
            np.testing.assert_allclose(acc, ref, rtol=1e-5)


@pytest.mark.parametrize("norm", [B.NORM_L1, B.NORM_LINF])
def test_allocation_from_another_criterion(norm):
    X = inputs.make_activations(2048, 768, inputs.BF16, 77, device="cuda")
    _, a = _gpu_norm(X, norm)
    bits, order = gpu_allocate(a, 2.6)
    ref_bits, ref_order = oracle.allocate_bits(a, 2.6)
    assert np.array_equal(bits, ref_bits) and np.array_equal(order, ref_order)


def test_unknown_norm_is_rejected():
    X = inputs.make_activations(64, 64, inputs.BF16, 1, device="cuda")
    acc = torch.zeros(64, dtype=torch.float64, device="cuda")
    with pytest.raises(B.CmpqError) as e:
        B.cmpq_collect_stats_norm(X, 3, acc, B.workspace(B.OP_COLLECT_STATS, 64))
    assert e.value.status == 1


@pytest.mark.parametrize("norm", [B.NORM_L2, B.NORM_L1, B.NORM_LINF])
@pytest.mark.parametrize("bad", [float("inf"), float("-inf"), float("nan")])
def test_nonfinite_activation_sets_the_flag_and_nothing_else_changes(norm, bad):
    """A NaN or an infinity among the activations: bit 0 of the caller's word is set (the reduction reads
    every value anyway) and every other column's statistic is what it would be without it."""
    X = inputs.make_activations(700, 512, inputs.BF16, 9, device="cuda")
    ws = B.workspace(B.OP_COLLECT_STATS, 512)
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    clean = torch.zeros(512, dtype=torch.float64, device="cuda")
    B.cmpq_collect_stats_norm(X, norm, clean, ws, nonfinite=flag)
    B.cmpq_check_finite(flag)                                   # finite input: no error
    assert int(flag.item()) == 0
    Xb = X.clone()
    Xb[123, 45] = bad
    acc = torch.zeros(512, dtype=torch.float64, device="cuda")
    B.cmpq_collect_stats_norm(Xb, norm, acc, ws, nonfinite=flag)
    with pytest.raises(B.CmpqError) as e:
        B.cmpq_check_finite(flag)
    assert e.value.status == 6 and int(flag.item()) == 1
    keep = torch.ones(512, dtype=torch.bool, device="cuda")
    keep[45] = False
    assert torch.equal(acc[keep], clean[keep])
    assert not torch.isfinite(acc[45])
    # without a word to report into, the call still runs
    B.cmpq_collect_stats_norm(Xb, norm, torch.zeros(512, dtype=torch.float64, device="cuda"), ws)
    torch.cuda.synchronize()


def test_bf16_square_beyond_fp32_is_reported_like_an_infinity():
    X = torch.zeros(64, 256, dtype=torch.bfloat16, device="cuda")
    X[3, 7] = 3.0e19                                            # finite in bf16, its square is not in fp32
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    acc = torch.zeros(256, dtype=torch.float64, device="cuda")
    B.cmpq_collect_stats(X, acc, B.workspace(B.OP_COLLECT_STATS, 256), nonfinite=flag)
    torch.cuda.synchronize()
    assert int(flag.item()) == 1
