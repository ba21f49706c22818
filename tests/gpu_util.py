"""Helpers for the GPU parity tests: run single C-ABI calls and return numpy results."""
import numpy as np
import torch

from paper_2410_13056_b200 import binding as B


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
