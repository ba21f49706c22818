"""Pins for the oracle's l1 and l_inf activation statistics (the paper's norm-ablation table compares
them with the default l2 norm as allocation criteria).  CPU only."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_13056_b200 import inputs


def _X(n=96, d_in=40, dtype=inputs.BF16, seed=4):
    X = inputs.make_activations(n, d_in, dtype, seed, n_outlier_channels=3)
    return X, inputs.as_u16(X)


@pytest.mark.parametrize("dtype", [inputs.F16, inputs.BF16])
def test_norms_against_numpy(dtype):
    X, Xu = _X(dtype=dtype)
    Xd = X.double().numpy()
    l1 = oracle.collect_stats_norm(Xu, dtype, oracle.NORM_L1)
    li = oracle.collect_stats_norm(Xu, dtype, oracle.NORM_LINF)
    l2 = oracle.collect_stats_norm(Xu, dtype, oracle.NORM_L2)
    assert np.allclose(l1, np.linalg.norm(Xd, ord=1, axis=0), rtol=1e-13)
    assert np.array_equal(li, np.linalg.norm(Xd, ord=np.inf, axis=0))          # a maximum is exact
    assert np.allclose(np.sqrt(l2), np.linalg.norm(Xd, ord=2, axis=0), rtol=1e-13)
    assert np.array_equal(l2, oracle.collect_stats(Xu, dtype))                   # norm 0 is the default statistic
    assert np.all(li <= l1 + 1e-300) and np.all(l1 <= np.sqrt(X.shape[0] * l2) * (1 + 1e-12))   # norm inequalities
    a1 = oracle.finalize_stats_norm(l1, oracle.NORM_L1)
    assert a1.dtype == np.float32 and np.array_equal(a1, l1.astype(np.float32))
    assert np.array_equal(oracle.finalize_stats_norm(l2, oracle.NORM_L2), oracle.finalize_stats(l2))


def test_closed_forms_and_chunking():
    dtype = inputs.F16
    n, d_in = 50, 6
    X = torch.zeros((n, d_in), dtype=torch.float16)
    X[:, 0] = -1.5                 # constant column: l1 = n |v|, l_inf = |v|
    X[7, 1] = 3.0                  # one entry
    X[:, 2] = torch.arange(n).half() - 20.0
    Xu = inputs.as_u16(X)
    l1 = oracle.collect_stats_norm(Xu, dtype, oracle.NORM_L1)
    li = oracle.collect_stats_norm(Xu, dtype, oracle.NORM_LINF)
    assert l1[0] == 1.5 * n and li[0] == 1.5 and l1[1] == 3.0 and li[1] == 3.0 and l1[3] == 0 and li[3] == 0
    assert l1[2] == sum(abs(t - 20) for t in range(n)) and li[2] == 29.0
    # accumulation over chunks of tokens gives the same statistic
    for norm in (oracle.NORM_L1, oracle.NORM_LINF):
        acc = oracle.collect_stats_norm(Xu[:13], dtype, norm)
        acc = oracle.collect_stats_norm(Xu[13:], dtype, norm, acc)
        assert np.array_equal(acc, oracle.collect_stats_norm(Xu, dtype, norm))
    # scaling by a power of two scales both norms exactly
    X2u = inputs.as_u16(X * 4)
    assert np.array_equal(oracle.collect_stats_norm(X2u, dtype, oracle.NORM_L1), 4 * l1)
    assert np.array_equal(oracle.collect_stats_norm(X2u, dtype, oracle.NORM_LINF), 4 * li)
