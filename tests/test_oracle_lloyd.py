"""Pins for the oracle's channel K-means (Section 3.2.1; quantizer of Section 3): exhaustive optimal
1-D clustering on tiny inputs, a library Lloyd from the same start, invariants and special cases."""
import itertools

import numpy as np
import pytest

import oracle


def _sse(x, lut, code):
    return float(((x.astype(np.float64) - lut[code].astype(np.float64)) ** 2).sum())


def _optimal_sse(x, K):
    """Exact optimum of 1-D K-means: clusters are contiguous runs of the sorted points, so try
    every way of cutting the sorted sequence into K non-empty runs (N <= 16)."""
    xs = np.sort(x.astype(np.float64))
    N = len(xs)
    K = min(K, N)
    best = np.inf
    for cuts in itertools.combinations(range(1, N), K - 1):
        edges = (0,) + cuts + (N,)
        s = 0.0
        for lo, hi in zip(edges[:-1], edges[1:]):
            seg = xs[lo:hi]
            s += ((seg - seg.mean()) ** 2).sum()
        best = min(best, s)
    return best


def _start(x, K):
    xs = np.sort(x)
    N = len(xs)
    return np.array([xs[((2 * k + 1) * N) // (2 * K)] for k in range(K)], np.float32)


# ----------------------------------------------------------------------------- start
def test_start_is_the_evenly_spaced_order_statistics():
    x = np.arange(16, dtype=np.float32)[::-1].copy()  # unsorted on purpose
    lut, code, err = oracle.lloyd(x, 4, 0)
    assert np.array_equal(lut[:4], [2, 6, 10, 14])   # hand-computed: ((2k+1)*16)//8
    assert np.all(lut[4:] == 0)
    # with T = 0 the codes are nearest-start codes, ties to the lower index
    assert np.array_equal(code[::-1], [0, 0, 0, 0, 0, 1, 1, 1, 1, 2, 2, 2, 2, 3, 3, 3])
    assert np.array_equal(err[::-1], [2, 1, 0, 1, 2, 1, 0, 1, 2, 1, 0, 1, 2, 1, 0, 1])


# ----------------------------------------------------------------------------- brute force
@pytest.mark.parametrize("K", [4, 8, 16])
@pytest.mark.parametrize("seed", range(6))
def test_tiny_inputs_against_exhaustive_optimum(K, seed):
    rng = np.random.default_rng(100 * K + seed)
    N = int(rng.integers(K, 13 if K == 4 else 17))
    if K == 8:
        N = min(N, 14)
    x = (rng.standard_normal(N) * 0.02).astype(np.float16).astype(np.float32)
    lut, code, err = oracle.lloyd(x, K, 50)
    opt = _optimal_sse(x, K)
    got = _sse(x, lut, code)
    assert got >= opt - 1e-12 - 1e-6 * opt
    # Lloyd's fixed point (T = 50 is far beyond convergence at this size)
    for k in range(K):
        members = x[code == k]
        if len(members):
            assert lut[k] == np.float32(members.astype(np.float64).sum() / len(members))
    d = np.abs(x[:, None] - lut[None, :K])
    assert np.array_equal(code, d.argmin(1))          # nearest, first minimum
    assert np.array_equal(err, d.min(1))
    if N == K and len(np.unique(x)) == N:
        assert got == 0.0


@pytest.mark.parametrize("K", [4, 8, 16])
def test_separated_clumps_reach_the_exhaustive_optimum(K):
    rng = np.random.default_rng(K)
    per = 16 // K if K < 16 else 1
    centres = np.arange(K) * 1.0 - K / 2
    x = np.concatenate([c + 0.01 * rng.standard_normal(per) for c in centres])
    x = x.astype(np.float16).astype(np.float32)
    rng.shuffle(x)
    lut, code, _ = oracle.lloyd(x, K, 5)
    assert _sse(x, lut, code) == pytest.approx(_optimal_sse(x, K), rel=1e-5, abs=1e-12)
    assert np.all(np.diff(lut[:K]) > 0)


# ----------------------------------------------------------------------------- library Lloyd
@pytest.mark.parametrize("K,T", [(4, 3), (8, 10), (16, 20), (8, 1)])
def test_against_sklearn_lloyd_from_the_same_start(K, T):
    from sklearn.cluster import KMeans

    rng = np.random.default_rng(7 + K)
    x = (rng.standard_normal(4096) * 0.02).astype(np.float32)
    x[rng.integers(0, 4096, 20)] += rng.standard_t(3, 20).astype(np.float32) * 0.1
    lut, code, err = oracle.lloyd(x, K, T)
    km = KMeans(n_clusters=K, init=_start(x, K).astype(np.float64).reshape(-1, 1), n_init=1,
                algorithm="lloyd", tol=0.0, max_iter=T)
    km.fit(x.astype(np.float64).reshape(-1, 1))
    assert km.n_iter_ == T  # it did not stop early, so it did exactly T updates as well
    ref = km.cluster_centers_.ravel()
    np.testing.assert_allclose(lut[:K], ref, rtol=2e-6, atol=1e-9)
    ref_code = np.abs(x[:, None].astype(np.float64) - ref[None, :]).argmin(1)
    assert np.count_nonzero(ref_code != code) <= 2   # only points within rounding of a boundary


# ----------------------------------------------------------------------------- invariants
@pytest.mark.parametrize("K", [4, 8, 16])
def test_sse_never_increases_and_centroids_stay_sorted(K):
    rng = np.random.default_rng(3 * K)
    x = (rng.standard_normal(2000) * 0.02).astype(np.float16).astype(np.float32)
    lut, code, err, sse = oracle.lloyd(x, K, 25, trace=True)
    assert np.all(np.diff(sse) <= 1e-9 * sse[0])
    assert np.all(np.diff(lut[:K]) > 0)
    assert sse[-1] == pytest.approx(float((err.astype(np.float64) ** 2).sum()), rel=1e-12)
    # more iterations can only help; T iterations are exactly T updates
    sse_by_T = [_sse(x, *oracle.lloyd(x, K, T)[:2]) for T in (0, 1, 2, 5)]
    np.testing.assert_allclose(sse_by_T, sse[[0, 1, 2, 5]], rtol=1e-6)  # trace squares fp32 distances


def test_special_cases():
    # constant channel: all codes 0, all centroids equal the value, zero error
    x = np.full(64, 0.125, np.float32)
    lut, code, err = oracle.lloyd(x, 8, 4)
    assert np.all(code == 0) and np.all(lut[:8] == 0.125) and np.all(err == 0)
    # all-zero channel (a removed O_act row); -0 and +0 are the same point
    x = np.zeros(32, np.float32)
    x[::2] = -0.0
    lut, code, err = oracle.lloyd(x, 16, 3)
    assert np.all(code == 0) and np.all(err == 0)
    assert np.all(lut.view(np.uint32) == 0)  # +0, not -0
    # two-valued channel, the start picks one value K-1 times: still zero error after 3 updates
    x = np.array([1.0] * 60 + [-3.0] * 4, np.float32)
    lut, code, err = oracle.lloyd(x, 4, 3)
    assert np.all(err == 0) and set(np.unique(lut[code])) == {1.0, -3.0}
    # an empty cluster keeps its centroid
    x = np.array([0.0] * 26 + [1.0] * 3 + [2.0] * 3, np.float32)
    lut0, _, _ = oracle.lloyd(x, 4, 0)
    lut5, code5, _ = oracle.lloyd(x, 4, 5)
    assert np.array_equal(lut0[:4], [0, 0, 0, 1])
    assert np.all(code5[:26] == 0) and np.all(code5[26:] == 3)
    assert lut5[1] == 0 and lut5[2] == 0          # clusters 1 and 2 never had members
    assert lut5[3] == 1.5
    # equal distances go to the lower index: x = 0.5 between centroids 0 and 1
    x = np.array([0.0, 0.0, 0.5, 1.0, 1.0, 1.0, 0.0, 0.0], np.float32)
    lut, code, _ = oracle.lloyd(x, 2, 0)  # K = 2 is outside the product's range but legal here
    assert np.array_equal(lut[:2], [0.0, 1.0]) and code[2] == 0


def test_constant_weights_change_nothing_and_weighted_means_hold():
    rng = np.random.default_rng(11)
    x = (rng.standard_normal(512) * 0.02).astype(np.float16).astype(np.float32)
    base = oracle.lloyd(x, 8, 30)
    same = oracle.lloyd(x, 8, 30, s=np.full(512, 2.0))
    assert np.array_equal(base[0], same[0]) and np.array_equal(base[1], same[1])
    s = rng.integers(1, 4, 512).astype(np.float64)
    lut, code, _ = oracle.lloyd(x, 8, 60, s=s)
    for k in range(8):
        m = code == k
        if m.any():
            assert lut[k] == np.float32((s[m] * x[m].astype(np.float64)).sum() / s[m].sum())
