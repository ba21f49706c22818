"""The allocation-free statistic entry point (for callers that cannot obtain device memory, such
as code running inside another framework's memory plan) against the regular entry point.

Collected last on purpose: a failure here must not hide the result of any other test."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_13056_b200 import binding as B
from paper_2410_13056_b200 import inputs

pytestmark = pytest.mark.gpu

STAT_RTOL = 1e-5   # the tolerance of the statistic everywhere else in this test suite


def _both(X):
    d_in = X.shape[1]
    ref = torch.zeros(d_in, dtype=torch.float64, device="cuda")
    B.cmpq_collect_stats(X, ref, B.workspace(B.OP_COLLECT_STATS, d_in))
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    got = torch.zeros(d_in, dtype=torch.float64, device="cuda")
    after_out = torch.cuda.memory_allocated()
    B.cmpq_collect_stats_static(X, got)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == after_out >= before   # the call itself took nothing from torch
    return got.cpu().numpy(), ref.cpu().numpy()


def test_static_scratch_matches_workspace_version_on_two_calls_in_a_row():
    # first call: a wide matrix, so the built-in array is filled with large partial sums
    X1 = inputs.make_activations(6000, 4096, inputs.BF16, 41, device="cuda")
    got1, ref1 = _both(X1)
    np.testing.assert_allclose(np.sqrt(got1), np.sqrt(ref1), rtol=STAT_RTOL)
    # and against the CPU checker's sums (fp64, token order), not only against the library's other entry
    np.testing.assert_allclose(got1, oracle.collect_stats(inputs.as_u16(X1), inputs.BF16), rtol=STAT_RTOL)
    # second call right after it: another shape and dtype, small values, ragged width (scalar
    # path); anything the first call left in the array must not leak into this result
    X2 = (inputs.make_activations(777, 1001, inputs.F16, 42, device="cuda").float() * 1e-3).to(torch.float16)
    got2, ref2 = _both(X2)
    np.testing.assert_allclose(np.sqrt(got2), np.sqrt(ref2), rtol=STAT_RTOL)
    np.testing.assert_allclose(got2, oracle.collect_stats(inputs.as_u16(X2), inputs.F16), rtol=STAT_RTOL)
    # and the first input again gives the first answer again, bit for bit
    got3, _ = _both(X1)
    assert np.array_equal(got3, got1)


def test_static_scratch_accumulates_and_rejects_what_does_not_fit():
    X = inputs.make_activations(300, 512, inputs.BF16, 43, device="cuda")
    s = torch.zeros(512, dtype=torch.float64, device="cuda")
    B.cmpq_collect_stats_static(X[:100], s)
    B.cmpq_collect_stats_static(X[100:], s)
    B.cmpq_collect_stats_static(X[:0], s)                 # empty chunk: nothing happens
    whole = torch.zeros(512, dtype=torch.float64, device="cuda")
    B.cmpq_collect_stats_static(X, whole)
    torch.cuda.synchronize()
    np.testing.assert_allclose(s.cpu().numpy(), whole.cpu().numpy(), rtol=1e-9)
    wide = torch.zeros(2, 32768 + 8, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(32768 + 8, dtype=torch.float64, device="cuda")
    with pytest.raises(B.CmpqError) as e:
        B.cmpq_collect_stats_static(wide, out)
    assert e.value.status == 2 and torch.all(out == 0)    # CMPQ_ERR_UNSUPPORTED, nothing written
    ok = torch.ones(3, 32768, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(32768, dtype=torch.float64, device="cuda")
    B.cmpq_collect_stats_static(ok, out)
    torch.cuda.synchronize()
    assert torch.all(out == 3.0)
