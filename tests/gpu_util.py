"""Helpers for the GPU parity tests: run single C-ABI calls and return numpy results."""
import numpy as np
import torch

import oracle
from paper_2410_13056_b200 import binding as B
from paper_2410_13056_b200 import inputs


def dev(arr, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(arr))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def gpu_stats(X, chunks=1):
    n, d_in = X.shape
    sumsq = torch.zeros(d_in, dtype=torch.float64, device="cuda")
    a = torch.empty(d_in, dtype=torch.float32, device="cuda")
    ws = B.workspace(B.OP_COLLECT_STATS, d_in)
    edges = np.linspace(0, n, chunks + 1).astype(int)
    for lo, hi in zip(edges[:-1], edges[1:]):
        B.cmpq_collect_stats(X[lo:hi], sumsq, ws)
    B.cmpq_finalize_stats(sumsq, a)
    torch.cuda.synchronize()
    return sumsq.cpu().numpy(), a.cpu().numpy()


def gpu_allocate(a_np, b, mode=B.ALLOC_RANK, want_order=True):
    a = dev(a_np)
    d_in = a.numel()
    bits = torch.empty(d_in, dtype=torch.uint8, device="cuda")
    order = torch.empty(d_in, dtype=torch.int32, device="cuda") if want_order else None
    B.cmpq_allocate_bits(a, b, mode, bits, order, B.workspace(B.OP_ALLOCATE_BITS, d_in))
    torch.cuda.synchronize()
    return bits.cpu().numpy(), (order.cpu().numpy() if want_order else None)


def gpu_extract(W, a_np, bits_np, n_act, n_q, T):
    d_in, d_out = W.shape
    nnz = n_act * d_out + n_q
    rows = torch.empty(nnz, dtype=torch.int32, device="cuda")
    cols = torch.empty(nnz, dtype=torch.int32, device="cuda")
    vals = torch.empty(nnz, dtype=torch.int16, device="cuda")
    B.cmpq_extract_outliers(W, dev(a_np), dev(bits_np), n_act, n_q, T, rows, cols, vals,
                            B.workspace(B.OP_EXTRACT_OUTLIERS, d_in, d_out))
    torch.cuda.synchronize()
    return rows.cpu().numpy(), cols.cpu().numpy(), vals.cpu().numpy().view(np.uint16)


def gpu_quantize(W, bits_np, rows_np, cols_np, T, sens=None):
    d_in, d_out = W.shape
    lut = torch.full((d_in, 16), -7.0, dtype=torch.float32, device="cuda")
    codes = torch.full((d_in, d_out), 255, dtype=torch.uint8, device="cuda")
    counters = torch.zeros(2, dtype=torch.int64, device="cuda")
    rows = dev(rows_np) if len(rows_np) else None
    cols = dev(cols_np) if len(cols_np) else None
    B.cmpq_quantize_layer(W, dev(bits_np), rows, cols, T, lut, codes,
                          B.workspace(B.OP_QUANTIZE_LAYER, d_in, d_out), sens=sens,
                          inexact_rows=counters[0:1].view(torch.int32)[0:1], sweeps=counters[1:2])
    torch.cuda.synchronize()
    c = counters.cpu().numpy()
    return lut.cpu().numpy(), codes.cpu().numpy(), int(c[0] & 0xffffffff), int(c[1])


def gpu_pack(codes_np, bits_np):
    d_in, d_out = codes_np.shape
    words = B.cmpq_packed_words(torch.from_numpy(np.ascontiguousarray(bits_np)), d_out)
    packed = torch.full((words + 8,), -1, dtype=torch.int32, device="cuda")
    row_off = torch.empty(d_in + 1, dtype=torch.int64, device="cuda")
    perm = torch.empty(d_in, dtype=torch.int32, device="cuda")
    seg = torch.empty(3, dtype=torch.int64, device="cuda")
    B.cmpq_pack(dev(codes_np), dev(bits_np), packed, row_off, perm, seg, B.workspace(B.OP_PACK, d_in, d_out))
    torch.cuda.synchronize()
    p = packed.cpu().numpy().view(np.uint32)
    assert np.all(p[words:] == 0xffffffff), "pack wrote past the end"
    return p[:words], row_off.cpu().numpy(), perm.cpu().numpy(), seg.cpu().numpy()


def result_arrays(r):
    """A LayerResult's buffers as host numpy arrays (16-bit values and packed words as unsigned)."""
    out = {k: getattr(r, k).cpu().numpy() for k in ("a", "bits", "rows", "cols", "lut", "row_off", "perm", "seg_rows")}
    out["vals"] = r.vals.cpu().numpy().view(np.uint16)
    out["packed"] = r.packed.cpu().numpy().view(np.uint32)
    if r.codes is not None:
        out["codes"] = r.codes.cpu().numpy()
    else:  # a pass that never materialised the byte codes: the checker's unpacker recovers them
        out["codes"] = oracle.unpack(out["packed"], out["row_off"], out["perm"], out["bits"], int(r.d_out))
    return out


def chain_with_gpu_statistic(Wu, dtype, a_gpu, b, n_act, n_q, T):
    """The checker's steps 2..8 fed with the statistic the GPU produced (the statistic itself is
    compared within tolerance; everything after it must then agree bit for bit)."""
    bits, _ = oracle.allocate_bits(a_gpu, b)
    rows, cols, vals = oracle.extract_outliers(Wu, dtype, a_gpu, bits, n_act, n_q, T)
    lut, codes = oracle.quantize_layer(Wu, dtype, bits, rows, cols, T)
    packed, row_off, perm, seg = oracle.pack(codes, bits)
    return dict(bits=bits, rows=rows, cols=cols, vals=vals, lut=lut, codes=codes, packed=packed,
                row_off=row_off, perm=perm, seg_rows=seg)


def assert_whole_layer_equal(g, ref):
    """Every output of the pass against the checker's, element by element (tables also bit for bit)."""
    for k, v in ref.items():
        if k == "lut":
            np.testing.assert_allclose(g[k], v, rtol=1e-4)
            assert np.array_equal(g[k].view(np.uint32), v.view(np.uint32)), k
        elif k != "a":
            assert np.array_equal(g[k], v), k


def check_statistic_columns(X, a_gpu, dtype, extra=()):
    """Sampled columns of the statistic against the checker (fp64, token order)."""
    d_in = X.shape[1]
    colsel = np.unique(np.array([0, 1, 7, 8, 255 % d_in, 256 % d_in, d_in // 2, d_in - 1] + list(extra)))
    Xs = X[:, torch.from_numpy(colsel).to(X.device)].contiguous()
    a_ref = oracle.finalize_stats(oracle.collect_stats(inputs.as_u16(Xs), dtype))
    np.testing.assert_allclose(a_gpu[colsel], a_ref, rtol=1e-5)


def check_layer_sampled(W, g, dtype, b, T, n_act, n_q, stripe=None):
    """Everything after the statistic of one full-size layer, from the GPU's own statistic g["a"]:
    allocation, outlier-list structure and packing in full; the provisional and the final fit on sampled
    channels.  stripe = (first, step): additionally EVERY channel first, first + step, ... is fitted by
    the checker, the kept entries of those channels must be exactly the ones their errors select, and
    codes and tables of all of them are compared."""
    d_in, d_out = W.shape
    Wu = inputs.as_u16(W)
    bits_ref, order_ref = oracle.allocate_bits(g["a"], b)
    assert np.array_equal(g["bits"], bits_ref)
    n2, n4 = oracle.alloc_counts(d_in, b)
    assert (g["bits"] == 2).sum() == n2 and (g["bits"] == 4).sum() == n4
    # outlier list: structure and O_act rows
    lin = g["rows"].astype(np.int64) * d_out + g["cols"]
    assert np.all(np.diff(lin) > 0)
    assert np.array_equal(g["vals"], Wu[g["rows"], g["cols"]])
    per_row = np.bincount(g["rows"], minlength=d_in)
    act_rows = np.sort(order_ref[d_in - n_act:])
    assert np.array_equal(np.flatnonzero(per_row == d_out), act_rows)
    assert per_row[per_row < d_out].sum() == n_q
    is_act = np.zeros(d_in, bool)
    is_act[act_rows] = True
    row_start = np.concatenate([[0], np.cumsum(per_row)])
    cols_of = lambda i: g["cols"][row_start[i]:row_start[i + 1]]
    def row_values(i):
        return W[i].float().cpu().numpy()

    # O_q: the provisional fit of sampled rows reproduces exactly the entries taken in those rows,
    # and no error left behind in a sampled row exceeds the smallest error taken in any sampled row
    sample = [i for i in (0, 1, 17, d_in // 8, d_in // 2, d_in - 1, int(np.argmax(per_row * ~is_act))) if not is_act[i]]
    if stripe is not None:
        sample = set(sample) | {i for i in range(stripe[0], d_in, stripe[1]) if not is_act[i]}
    sample = sorted(set(sample))
    taken_min, left_max = np.inf, 0.0
    tie_taken_last, tie_left_first = -1, None
    errs = {}
    for i in sample:
        _, _, err = oracle.lloyd(row_values(i), 1 << int(bits_ref[i]), T)
        errs[i] = err
        mask = np.zeros(d_out, bool)
        mask[cols_of(i)] = True
        if mask.any():
            taken_min = min(taken_min, err[mask].min())
            assert err[mask].min() >= err[~mask].max(), i
        if not mask.all():
            left_max = max(left_max, err[~mask].max())
    assert left_max <= taken_min
    if n_q > 0 and np.isfinite(taken_min):
        # entries whose error equals the smallest one taken: the kept ones come first in linear-index order
        for i in sample:
            mask = np.zeros(d_out, bool)
            mask[cols_of(i)] = True
            tie = errs[i] == np.float32(taken_min)
            if (tie & mask).any():
                tie_taken_last = max(tie_taken_last, i * d_out + int(np.flatnonzero(tie & mask).max()))
            if (tie & ~mask).any():
                first = i * d_out + int(np.flatnonzero(tie & ~mask).min())
                tie_left_first = first if tie_left_first is None else min(tie_left_first, first)
            # every error above the threshold of the sampled rows is kept, none below it
            assert mask[errs[i] > np.float32(taken_min)].all() and not mask[errs[i] < np.float32(taken_min)].any(), i
        assert tie_left_first is None or tie_taken_last < tie_left_first
    # final fit: sampled channels (every width present, an O_act row, the row with most O_q entries)
    sample2 = sample + ([int(act_rows[0])] if n_act else []) + [
        int(np.flatnonzero(bits_ref == c)[k]) for c in (2, 3, 4) for k in (0, -1) if (bits_ref == c).any()]
    if stripe is not None:
        sample2 += [i for i in range(stripe[0], d_in, stripe[1]) if is_act[i]]
    for i in sorted(set(sample2)):
        xi = row_values(i)
        xi[cols_of(i)] = 0
        lut, code, _ = oracle.lloyd(xi, 1 << int(bits_ref[i]), T)
        assert np.array_equal(code, g["codes"][i]), i
        np.testing.assert_allclose(g["lut"][i], lut, rtol=1e-4)
        assert np.array_equal(g["lut"][i].view(np.uint32), lut.view(np.uint32)), i
    assert np.all(g["codes"] < (1 << g["bits"].astype(np.int64))[:, None])
    # packing: full comparison against the checker's packer
    packed, row_off, perm, seg = oracle.pack(g["codes"], g["bits"])
    assert np.array_equal(g["packed"], packed) and np.array_equal(g["row_off"], row_off)
    assert np.array_equal(g["perm"], perm) and np.array_equal(g["seg_rows"], seg)
    return len(sample), len(set(sample2))
