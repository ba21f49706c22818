"""GPU parity of the whole pass (the chain of C-ABI calls) on the small workload in full and on
the Llama-shaped workloads through samples and properties that hold at any size."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_13056_b200 import binding as B
from paper_2410_13056_b200 import inputs
from paper_2410_13056_b200.pipeline import LayerQuantizer

pytestmark = pytest.mark.gpu


def _np(r):
    out = {k: getattr(r, k).cpu().numpy() for k in ("a", "bits", "rows", "cols", "lut", "codes", "row_off",
                                                     "perm", "seg_rows")}
    out["vals"] = r.vals.cpu().numpy().view(np.uint16)
    out["packed"] = r.packed.cpu().numpy().view(np.uint32)
    return out


def _chain_with_gpu_statistic(Wu, dtype, a_gpu, b, n_act, n_q, T):
    """The checker's steps 2..8 fed with the statistic the GPU produced (the statistic itself is
    compared within tolerance; everything after it must then agree bit for bit)."""
    bits, _ = oracle.allocate_bits(a_gpu, b)
    rows, cols, vals = oracle.extract_outliers(Wu, dtype, a_gpu, bits, n_act, n_q, T)
    lut, codes = oracle.quantize_layer(Wu, dtype, bits, rows, cols, T)
    packed, row_off, perm, seg = oracle.pack(codes, bits)
    return dict(bits=bits, rows=rows, cols=cols, vals=vals, lut=lut, codes=codes, packed=packed,
                row_off=row_off, perm=perm, seg_rows=seg)


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


def _sampled_parity(cfg_name, layer_index, b):
    """One full-size layer through the quantizer in the launch configuration the benchmark uses; the
    checker verifies sampled channels and properties that hold at any size instead of re-running
    everything (a full single-threaded run would take minutes)."""
    cfg = inputs.CONFIGS[cfg_name]
    L = cfg.layers[layer_index]
    T = cfg.lloyd_iters
    d_in, d_out = L.d_in, L.d_out
    seed = inputs.layer_seed(cfg, layer_index)
    W = inputs.make_weight(d_in, d_out, cfg.dtype, seed, device="cuda")
    X = inputs.make_activations(cfg.n_tokens, d_in, cfg.dtype, seed, device="cuda")
    q = LayerQuantizer(d_in, d_out)
    r = q.run(X, W, b, T)
    g = _np(r)
    assert int(q.counters[0].item()) == 0
    assert (q.n_act, q.n_q) == oracle.default_counts(d_in, d_out)
    # statistic: sampled columns against the checker (fp64, token order)
    colsel = np.unique(np.array([0, 1, 7, 8, 255, 256, d_in // 2, d_in - 1] + list(np.argsort(g["a"])[-4:])))
    Xs = X[:, torch.from_numpy(colsel).cuda()].contiguous()
    a_ref = oracle.finalize_stats(oracle.collect_stats(inputs.as_u16(Xs), cfg.dtype))
    np.testing.assert_allclose(g["a"][colsel], a_ref, rtol=1e-5)
    del X, Xs
    # allocation: exact, from the GPU statistic
    bits_ref, order_ref = oracle.allocate_bits(g["a"], b)
    assert np.array_equal(g["bits"], bits_ref)
    n2, n4 = oracle.alloc_counts(d_in, b)
    assert (g["bits"] == 2).sum() == n2 and (g["bits"] == 4).sum() == n4
    # outlier list: structure and O_act rows
    lin = g["rows"].astype(np.int64) * d_out + g["cols"]
    assert np.all(np.diff(lin) > 0)
    Wu = inputs.as_u16(W)
    assert np.array_equal(g["vals"], Wu[g["rows"], g["cols"]])
    per_row = np.bincount(g["rows"], minlength=d_in)
    act_rows = np.sort(order_ref[d_in - q.n_act:])
    assert np.array_equal(np.flatnonzero(per_row == d_out), act_rows)
    assert per_row[per_row < d_out].sum() == q.n_q
    # O_q: the provisional fit of sampled rows reproduces exactly the entries taken in those rows,
    # and no error left behind in a sampled row exceeds the smallest error taken in any sampled row
    is_act = np.zeros(d_in, bool)
    is_act[act_rows] = True
    sample = [i for i in (0, 1, 17, d_in // 8, d_in // 2, d_in - 1, int(np.argmax(per_row * ~is_act))) if not is_act[i]]
    taken_min, left_max = np.inf, 0.0
    for i in sample:
        xi = W[i].float().cpu().numpy()
        _, _, err = oracle.lloyd(xi, 1 << int(bits_ref[i]), T)
        mask = np.zeros(d_out, bool)
        mask[g["cols"][g["rows"] == i]] = True
        if mask.any():
            taken_min = min(taken_min, err[mask].min())
            assert err[mask].min() >= err[~mask].max()
        left_max = max(left_max, err[~mask].max())
    assert left_max <= taken_min
    # final fit: sampled channels (every width present, an O_act row, the row with most O_q entries)
    sample2 = sample + [int(act_rows[0])] + [int(np.flatnonzero(bits_ref == c)[k]) for c in (2, 3, 4)
                                              for k in (0, -1) if (bits_ref == c).any()]
    for i in sample2:
        xi = W[i].float().cpu().numpy()
        xi[g["cols"][g["rows"] == i]] = 0
        lut, code, _ = oracle.lloyd(xi, 1 << int(bits_ref[i]), T)
        assert np.array_equal(code, g["codes"][i]), i
        np.testing.assert_allclose(g["lut"][i], lut, rtol=1e-4)
        assert np.array_equal(g["lut"][i].view(np.uint32), lut.view(np.uint32)), i
    assert np.all(g["codes"] < (1 << g["bits"].astype(np.int64))[:, None])
    # packing: full comparison against the checker's packer
    packed, row_off, perm, seg = oracle.pack(g["codes"], g["bits"])
    assert np.array_equal(g["packed"], packed) and np.array_equal(g["row_off"], row_off)
    assert np.array_equal(g["perm"], perm) and np.array_equal(g["seg_rows"], seg)
    return g, q


def test_llama_attention_shape_sampled_parity():
    """The benchmark's workload shape (4096 x 4096 bf16, 131072 tokens, 20 iterations) at its own 2.2-bit
    budget and at the metric's 3.0 bits."""
    g, q = _sampled_parity("c2_attn7b", 0, 2.2)
    assert (q.n_act, q.n_q, q.nnz) == (18, 8388, 82116)
    assert (g["bits"] == 2).sum() == 3277 and g["packed"].nbytes == 4613632
    g, q = _sampled_parity("c2_attn7b", 0, 3.0)
    assert g["packed"].nbytes == 4096 * 4096 * 3 // 8


@pytest.mark.parametrize("layer_index,b", [(0, 2.5), (1, 3.5)])
def test_llama_mlp_shapes_sampled_parity(layer_index, b):
    """4096 x 11008 (up) and 11008 x 4096 (down) with 131072 calibration tokens."""
    g, q = _sampled_parity("c3_mlp7b", layer_index, b)
    assert q.nnz == (220688 if layer_index == 0 else 223248)


@pytest.mark.parametrize("layer_index", [0, 1])
def test_llama70b_mlp_shapes_sampled_parity(layer_index):
    """8192 x 28672 and 28672 x 8192 with 65536 calibration tokens at 2.5 bits."""
    g, q = _sampled_parity("c5_mlp70b", layer_index, 2.5)
    assert q.nnz == (1149632 if layer_index == 0 else 1174208)
    assert g["packed"].nbytes == 8192 * 28672 * 5 // 16


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


def test_budget_sweep_shares_the_statistic():
    """run_budgets computes the statistic once; every budget's outputs equal those of a separate pass."""
    d_in, d_out, n, T = 192, 640, 1024, 6
    W = inputs.make_weight(d_in, d_out, inputs.BF16, 61, device="cuda")
    X = inputs.make_activations(n, d_in, inputs.BF16, 61, device="cuda")
    budgets = [2.0, 2.5, 3.0, 3.5, 4.0]
    q = LayerQuantizer(d_in, d_out)
    got = {}
    q.run_budgets(X, W, budgets, T, on_result=lambda b, r: got.__setitem__(b, {k: v.copy() for k, v in _np(r).items()}))
    q2 = LayerQuantizer(d_in, d_out)
    for b in budgets:
        sep = _np(q2.run(X, W, b, T))
        for k in sep:
            assert np.array_equal(got[b][k], sep[k]), (b, k)
