"""Whole-layer parity at full size: the pass exactly as the benchmark launches it (graph replay,
outlier protection and final fit in one call) against the CPU checker, element by element, and the
32-block stack through the stack driver.

The checker needs about ten seconds for a 4096 x 4096 layer and half a minute for a 4096 x 11008 one,
so these are the slowest tests of the suite."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_13056_b200 import inputs
from paper_2410_13056_b200.pipeline import LayerQuantizer, StackQuantizer

from gpu_util import (assert_whole_layer_equal, chain_with_gpu_statistic, check_layer_sampled,
                      check_statistic_columns, result_arrays)

pytestmark = pytest.mark.gpu


def _whole_layer(cfg_name, layer_index, budgets, whole_statistic):
    cfg = inputs.CONFIGS[cfg_name]
    L = cfg.layers[layer_index]
    seed = inputs.layer_seed(cfg, layer_index)
    W = inputs.make_weight(L.d_in, L.d_out, cfg.dtype, seed, device="cuda")
    X = inputs.make_activations(cfg.n_tokens, L.d_in, cfg.dtype, seed, device="cuda")
    q = LayerQuantizer(L.d_in, L.d_out, keep_codes=False)   # as the benchmark: packed words only, no byte codes
    Wu = inputs.as_u16(W)
    for k, b in enumerate(budgets):
        q.run_graphed(X, W, b, cfg.lloyd_iters)            # captures
        g = result_arrays(q.run_graphed(X, W, b, cfg.lloyd_iters))   # a replay, as the benchmark times it
        assert int(q.counters[0].item()) == 0                 # no channel with inexact sums
        if k == 0:
            if whole_statistic:                               # all d_in columns, all tokens, fp64 in token order
                a_ref = oracle.finalize_stats(oracle.collect_stats(inputs.as_u16(X), cfg.dtype))
                np.testing.assert_allclose(g["a"], a_ref, rtol=1e-5)
            else:
                check_statistic_columns(X, g["a"], cfg.dtype, extra=list(np.argsort(g["a"])[-4:]))
        ref = chain_with_gpu_statistic(Wu, cfg.dtype, g["a"], b, q.n_act, q.n_q, cfg.lloyd_iters)
        assert_whole_layer_equal(g, ref)
    return q


def test_benchmark_path_whole_layer_attention_shape():
    """4096 x 4096 bf16, 131072 tokens, 20 iterations at the metric's 3.0 bits and at the workload's own
    2.2 bits: bits, the complete outlier list, every code, every table entry, the packed words."""
    q = _whole_layer("c2_attn7b", 0, [3.0, 2.2], whole_statistic=True)
    assert (q.n_act, q.n_q, q.nnz) == (18, 8388, 82116)


def test_benchmark_path_whole_layer_mlp_up_shape():
    """4096 x 11008 bf16 (the MLP up projection) at 3.0 bits, in full."""
    q = _whole_layer("c3_mlp7b", 0, [3.0], whole_statistic=False)
    assert q.nnz == 220688


def test_stack_driver_blocks_against_the_checker():
    """The 32-block stack (4 attention, 2 up/gate, 1 down projection per block, own seeded weights per
    layer, 3.0 bits) through StackQuantizer: the 21 layers of blocks 0, 15 and 31 are checked the way the
    single full-size layers are (sampled channels, everything else in full), and a further block gives the
    same bytes when it is quantized twice."""
    cfg = inputs.CONFIGS["c4_stack7b"]
    b, T = cfg.budgets[0], cfg.lloyd_iters
    src = inputs.StackInputs(cfg)
    per_block = len(cfg.layers)
    assert len(src.layers) == 224
    wanted = [blk * per_block + i for blk in (0, 15, 31) for i in range(per_block)]
    twice = [7 * per_block + i for i in range(per_block)]

    class Subset(StackQuantizer):          # the driver itself, restricted to the layers under test
        def __init__(self, keep):
            super().__init__(src.shapes())
            self.mine = [k for k in self.mine if k in keep]

    checked = []

    def check(k, r):
        g = result_arrays(r)
        assert int(r.inexact_rows.item()) == 0
        X, W = src.activations(src.layers[k][2].d_in), src.weights(src.shapes()[k])
        if k in wanted[:per_block]:        # the statistic of each width once per distinct input (X is shared)
            check_statistic_columns(X, g["a"], cfg.dtype)
        q = stack.quantizer(k)
        check_layer_sampled(W, g, cfg.dtype, b, T, q.n_act, q.n_q)
        checked.append(k)

    stack = Subset(set(wanted))
    out = stack.run(src, b, T, on_result=check)
    assert checked == wanted and out["layers"] == 21
    assert out["params"] == 3 * (4 * 4096 * 4096 + 3 * 4096 * 11008)

    runs = []
    for _ in range(2):
        got = {}
        stack2 = Subset(set(twice))
        stack2._quantizers = stack._quantizers     # same buffers: the second run overwrites the first
        stack2.run(src, b, T, on_result=lambda k, r: got.__setitem__(k, result_arrays(r)))
        runs.append(got)
    for k in twice:
        for name in runs[0][k]:
            assert np.array_equal(runs[0][k][name], runs[1][k][name]), (k, name)
    # layers of one shape differ from each other (own seeds), so the driver did not reuse stale inputs
    assert not np.array_equal(runs[0][twice[0]]["codes"], runs[0][twice[1]]["codes"])


def test_stack_driver_timed_run_reports_every_shape():
    cfg = inputs.CONFIGS["c4_stack7b"]
    src = inputs.StackInputs(cfg)
    stack = StackQuantizer(src.shapes()[:7])       # one block
    out = stack.run(src, 3.0, cfg.lloyd_iters, timed=True)
    assert out["layers"] == 7 and set(out["ms_by_shape"]) == {(4096, 4096), (4096, 11008), (11008, 4096)}
    assert 0 < out["ms"] < 1000
