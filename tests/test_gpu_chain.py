"""GPU parity of the whole pass (the chain of C-ABI calls) on the small workload in full and on
the Llama-shaped workloads through samples and properties that hold at any size."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_13056_b200 import binding as B
from paper_2410_13056_b200 import inputs
from paper_2410_13056_b200.pipeline import LayerQuantizer

from gpu_util import (assert_whole_layer_equal, chain_with_gpu_statistic, check_layer_sampled,
                      check_statistic_columns, result_arrays)

pytestmark = pytest.mark.gpu


_np = result_arrays
_chain_with_gpu_statistic = chain_with_gpu_statistic


@pytest.fixture(params=["ordered", "all_pairs"])
def assignment(request):
    B.cmpq_set_lloyd_assignment(B.ASSIGN_ALL_PAIRS if request.param == "all_pairs" else B.ASSIGN_ORDERED)
    yield request.param
    B.cmpq_set_lloyd_assignment(B.ASSIGN_ORDERED)


def test_small_workload_full_parity(assignment):
    cfg = inputs.CONFIGS["c1_small"]
    L = cfg.layers[0]
    W = inputs.make_weight(L.d_in, L.d_out, cfg.dtype, cfg.seed, device="cuda")
    X = inputs.make_activations(cfg.n_tokens, L.d_in, cfg.dtype, cfg.seed, device="cuda",
                                n_outlier_channels=cfg.n_outlier_channels)
    q = LayerQuantizer(L.d_in, L.d_out)
    assert (q.n_act, q.n_q, q.nnz) == (2, 131, 1155)
    g = _np(q.run(X, W, 3.0, cfg.lloyd_iters))
    Xu, Wu = inputs.as_u16(X), inputs.as_u16(W)
    ref = oracle.layer_pass(Xu, Wu, cfg.dtype, 3.0, q.n_act, q.n_q, cfg.lloyd_iters)
    np.testing.assert_allclose(g["a"], ref["a"], rtol=1e-5)
    for k in ("bits", "rows", "cols", "vals", "codes", "packed", "row_off", "perm", "seg_rows"):
        assert np.array_equal(g[k], ref[k]), k
    np.testing.assert_allclose(g["lut"], ref["lut"], rtol=1e-4)
    assert g["packed"].nbytes == 98304 and int(q.counters[0].item()) == 0
    # reconstruction error ||X (W - What)||_F: both sides evaluated by the checker in fp64
    Eg = oracle.recon_error(Xu, Wu, cfg.dtype, g["lut"], g["codes"], g["rows"], g["cols"], g["vals"])
    Er = oracle.recon_error(Xu, Wu, cfg.dtype, ref["lut"], ref["codes"], ref["rows"], ref["cols"], ref["vals"])
    assert Eg == pytest.approx(Er, rel=1e-4)
    # and on the device in fp32 from the library's own outputs
    What = torch.gather(q.lut, 1, q.codes.long())
    What[q.rows.long(), q.cols.long()] += W[q.rows.long(), q.cols.long()].float()
    E32 = torch.linalg.norm(X.float() @ (W.float() - What)).item()
    assert E32 == pytest.approx(Er, rel=1e-4)
    # a second run gives the same bytes
    g2 = _np(q.run(X, W, 3.0, cfg.lloyd_iters))
    for k in g:
        assert np.array_equal(g[k], g2[k]), k


@pytest.mark.parametrize("b", [2.0, 2.2, 3.0, 3.5, 4.0])
def test_midsize_layer_all_budgets(b):
    d_in, d_out, n, T = 256, 1536, 2048, 12
    W = inputs.make_weight(d_in, d_out, inputs.BF16, 31, device="cuda")
    X = inputs.make_activations(n, d_in, inputs.BF16, 31, device="cuda")
    q = LayerQuantizer(d_in, d_out)
    g = _np(q.run(X, W, b, T))
    Xu, Wu = inputs.as_u16(X), inputs.as_u16(W)
    a_ref = oracle.finalize_stats(oracle.collect_stats(Xu, inputs.BF16))
    np.testing.assert_allclose(g["a"], a_ref, rtol=1e-5)
    ref = _chain_with_gpu_statistic(Wu, inputs.BF16, g["a"], b, q.n_act, q.n_q, T)
    for k, v in ref.items():
        if k == "lut":
            np.testing.assert_allclose(g[k], v, rtol=1e-4)
        else:
            assert np.array_equal(g[k], v), k
    assert abs(g["bits"].mean() - b) <= 0.5 / d_in or b == 3.0


def _sampled_parity(cfg_name, layer_index, budgets, stripe=None, graphed=False):
    """One full-size layer through the quantizer in the launch configuration the benchmark uses, at every
    budget given (the statistic is checked once); the checker verifies sampled channels and properties
    that hold at any size instead of re-running everything (a full single-threaded run takes minutes)."""
    cfg = inputs.CONFIGS[cfg_name]
    L = cfg.layers[layer_index]
    T = cfg.lloyd_iters
    d_in, d_out = L.d_in, L.d_out
    seed = inputs.layer_seed(cfg, layer_index)
    W = inputs.make_weight(d_in, d_out, cfg.dtype, seed, device="cuda")
    X = inputs.make_activations(cfg.n_tokens, d_in, cfg.dtype, seed, device="cuda")
    q = LayerQuantizer(d_in, d_out)
    assert (q.n_act, q.n_q) == oracle.default_counts(d_in, d_out)
    out = {}
    for k, b in enumerate(budgets):
        r = (q.run_graphed if graphed else q.run)(X, W, b, T)
        g = _np(r)
        assert int(q.counters[0].item()) == 0
        if k == 0:
            check_statistic_columns(X, g["a"], cfg.dtype, extra=list(np.argsort(g["a"])[-4:]))
        check_layer_sampled(W, g, cfg.dtype, b, T, q.n_act, q.n_q, stripe=stripe)
        out[b] = g
    return out, q


def test_llama_attention_shape_sampled_parity():
    """The benchmark's workload shape (4096 x 4096 bf16, 131072 tokens, 20 iterations) at its own 2.2-bit
    budget and at the metric's 3.0 bits, eager calls (the graph-replayed path is compared in full in
    test_gpu_full_parity.py)."""
    out, q = _sampled_parity("c2_attn7b", 0, [2.2, 3.0])
    assert (q.n_act, q.n_q, q.nnz) == (18, 8388, 82116)
    assert (out[2.2]["bits"] == 2).sum() == 3277 and out[2.2]["packed"].nbytes == 4613632
    assert out[3.0]["packed"].nbytes == 4096 * 4096 * 3 // 8


@pytest.mark.parametrize("layer_index,budgets", [(0, [2.0, 2.5, 3.5, 4.0]), (1, [2.0, 2.5, 3.0, 3.5, 4.0])])
def test_llama_mlp_shapes_sampled_parity(layer_index, budgets):
    """4096 x 11008 (up) and 11008 x 4096 (down) with 131072 calibration tokens, every budget of the sweep
    (the up projection at 3.0 bits is compared in full in test_gpu_full_parity.py)."""
    out, q = _sampled_parity("c3_mlp7b", layer_index, budgets)
    assert q.nnz == (220688 if layer_index == 0 else 223248)
    for b, g in out.items():
        assert g["packed"].nbytes == round(4096 * 11008 * b / 8)


@pytest.mark.parametrize("layer_index", [0, 1])
def test_llama70b_mlp_shapes_striped_parity(layer_index):
    """8192 x 28672 and 28672 x 8192 with 65536 calibration tokens at 2.5 bits: every sixteenth channel is
    fitted by the checker (provisional and final fit), and the entries kept in those channels must be
    exactly the ones their errors select."""
    out, q = _sampled_parity("c5_mlp70b", layer_index, [2.5], stripe=(5, 16))
    assert q.nnz == (1149632 if layer_index == 0 else 1174208)
    assert out[2.5]["packed"].nbytes == 8192 * 28672 * 5 // 16


def test_graph_replay_gives_the_same_bytes_as_the_eager_pass():
    d_in, d_out, n, T = 192, 1024, 1024, 8
    W = inputs.make_weight(d_in, d_out, inputs.BF16, 7, device="cuda")
    X = inputs.make_activations(n, d_in, inputs.BF16, 7, device="cuda")
    q = LayerQuantizer(d_in, d_out)
    eager = _np(q.run(X, W, 2.5, T))
    first = _np(q.run_graphed(X, W, 2.5, T))       # captures, then replays once
    W2 = inputs.make_weight(d_in, d_out, inputs.BF16, 8, device="cuda")
    W.copy_(W2)                                       # same address, new contents
    replay = _np(q.run_graphed(X, W, 2.5, T))
    again = _np(q.run(X, W, 2.5, T))
    for k in eager:
        assert np.array_equal(eager[k], first[k]), k
        assert np.array_equal(replay[k], again[k]), k
    assert not np.array_equal(eager["codes"], replay["codes"])


@pytest.mark.parametrize("keep_codes", [True, False])
def test_tables_built_on_a_second_stream_give_the_same_bytes(keep_codes):
    """overlap_tables: the value tables are counted on a second stream while the statistic runs; eager and
    replayed from a graph, with new weights at the same address and with a budget change in between, every
    output equals the plain pass's (and hence the checker's, which the plain pass is compared with above)."""
    d_in, d_out, n, T = 200, 1536, 1024, 8
    W = inputs.make_weight(d_in, d_out, inputs.BF16, 17, device="cuda")
    X = inputs.make_activations(n, d_in, inputs.BF16, 17, device="cuda")
    plain, over = LayerQuantizer(d_in, d_out, keep_codes=keep_codes), LayerQuantizer(d_in, d_out, keep_codes=keep_codes)
    for step, b in enumerate([3.0, 2.3, 3.0]):
        if step == 2:
            W.copy_(inputs.make_weight(d_in, d_out, inputs.BF16, 18, device="cuda"))   # same address, new contents
        ref = _np(plain.run(X, W, b, T))
        eager = _np(over.run(X, W, b, T, overlap_tables=True))
        graphed = _np(over.run_graphed(X, W, b, T, overlap_tables=True))
        replay = _np(over.run_graphed(X, W, b, T, overlap_tables=True))
        for k in ref:
            assert np.array_equal(ref[k], eager[k]), (step, k)
            assert np.array_equal(ref[k], graphed[k]), (step, k)
            assert np.array_equal(ref[k], replay[k]), (step, k)
        assert int(over.counters[0].item()) == int(plain.counters[0].item())


@pytest.mark.parametrize("d_in,d_out,n,T,budgets", [
    (192, 640, 1024, 6, [2.0, 2.5, 3.0, 3.5, 4.0]),
    (300, 2048, 512, 9, [3.5, 2.5, 3.5, 2.0, 3.0, 2.5]),      # budgets revisited: every fit comes from the cache
    (64, 6000, 256, 4, [4.0, 3.0, 2.2]),
])
def test_budget_sweep_shares_statistic_tables_and_fits(d_in, d_out, n, T, budgets, assignment):
    """run_budgets computes the statistic and the value tables once and keeps the provisional fits per
    (channel, width); every budget's outputs equal those of a separate pass bit for bit, and those of the
    checker fed the same statistic."""
    W = inputs.make_weight(d_in, d_out, inputs.BF16, 61, device="cuda")
    X = inputs.make_activations(n, d_in, inputs.BF16, 61, device="cuda")
    q = LayerQuantizer(d_in, d_out)
    got = []
    q.run_budgets(X, W, budgets, T, on_result=lambda b, r: got.append({k: v.copy() for k, v in _np(r).items()}))
    q2 = LayerQuantizer(d_in, d_out)
    Wu = inputs.as_u16(W)
    for b, g in zip(budgets, got):
        sep = _np(q2.run(X, W, b, T))
        for k in sep:
            assert np.array_equal(g[k], sep[k]), (b, k)
        assert_whole_layer_equal(g, _chain_with_gpu_statistic(Wu, inputs.BF16, g["a"], b, q.n_act, q.n_q, T))
    # a sweep after the weights changed starts from a fresh cache (cmpq_sweep_begin): no stale fit is reused
    W2 = inputs.make_weight(d_in, d_out, inputs.BF16, 62, device="cuda")
    got2 = []
    q.run_budgets(X, W2, budgets[:2], T, on_result=lambda b, r: got2.append({k: v.copy() for k, v in _np(r).items()}))
    for b, g in zip(budgets[:2], got2):
        sep = _np(q2.run(X, W2, b, T))
        for k in sep:
            assert np.array_equal(g[k], sep[k]), (b, k)


def test_sweep_cache_with_another_iteration_count_is_bypassed_not_trusted():
    d_in, d_out, n = 96, 1024, 512
    W = inputs.make_weight(d_in, d_out, inputs.BF16, 63, device="cuda")
    X = inputs.make_activations(n, d_in, inputs.BF16, 63, device="cuda")
    q = LayerQuantizer(d_in, d_out)
    q.run_budgets(X, W, [3.0], 3)                       # leaves fits made with 3 iterations in the cache
    g = _np(q.run(X, W, 3.0, 8, reuse_statistic=True, sweep_cache=q._sweep_cache))
    sep = _np(LayerQuantizer(d_in, d_out).run(X, W, 3.0, 8))
    for k in sep:
        assert np.array_equal(g[k], sep[k]), k
