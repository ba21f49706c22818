"""Thin ctypes binding of the C ABI in include/cmpq.h.

Argument marshalling only: every step of the pass runs in the CUDA library.  Tensors are
torch CUDA tensors (torch is used for device memory and streams, nothing else); each function
has the name and the argument order of its C counterpart, enqueues work on the current torch
stream and raises CmpqError when the library returns a non-zero status.  There is no CPU
fallback: if libcmpq.so is missing or does not load, the first call raises.
"""
import ctypes
import os

import torch

F16, BF16 = 0, 1
ALLOC_RANK, ALLOC_QUANTILE = 0, 1
NORM_L2, NORM_L1, NORM_LINF = 0, 1, 2
ASSIGN_ORDERED, ASSIGN_ALL_PAIRS = 0, 1
(OP_COLLECT_STATS, OP_ALLOCATE_BITS, OP_EXTRACT_OUTLIERS, OP_QUANTIZE_LAYER, OP_PACK, OP_PROTECT_AND_QUANTIZE,
 OP_OUTLIERS_BY_COLUMN, OP_MATVEC, OP_QUANTIZE_LAYER_PACKED, OP_PROTECT_QUANTIZE_PACK) = range(10)
LUT_STRIDE = 16

EXPORTS = (
    "cmpq_collect_stats", "cmpq_collect_stats_static", "cmpq_finalize_stats", "cmpq_allocate_bits", "cmpq_extract_outliers",
    "cmpq_quantize_layer", "cmpq_pack", "cmpq_workspace_bytes", "cmpq_alloc_counts",
    "cmpq_default_counts", "cmpq_packed_words", "cmpq_status_string",
    "cmpq_set_lloyd_assignment", "cmpq_get_lloyd_assignment", "cmpq_lloyd_phase_events",
    "cmpq_protect_and_quantize", "cmpq_matvec", "cmpq_outliers_by_column",
    "cmpq_collect_stats_norm", "cmpq_finalize_stats_norm", "cmpq_transpose16",
    "cmpq_alu_probe", "cmpq_kernel_resources",
    "cmpq_sweep_cache_bytes", "cmpq_sweep_begin", "cmpq_sweep_budget", "cmpq_sweep_budget_pack",
    "cmpq_quantize_layer_packed", "cmpq_protect_quantize_pack", "cmpq_check_finite",
    "cmpq_matvec_f16lut", "cmpq_lut_bytes", "cmpq_store_lut", "cmpq_load_lut", "cmpq_table_bits_per_weight",
)

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libcmpq.so")
_lib = None


class CmpqError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        msg = lib().cmpq_status_string(self.status).decode()
        super().__init__("%s failed: %s (status %d)" % (where, msg, self.status))


def lib():
    """Loads libcmpq.so once; raises if it was not built (run paper_2410_13056_b200/build.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError("CUDA library %s is missing: build it with "
                               "`python -m paper_2410_13056_b200.build`" % _LIB_PATH)
        L = ctypes.CDLL(_LIB_PATH)
        i64, vp, dbl, sz = ctypes.c_int64, ctypes.c_void_p, ctypes.c_double, ctypes.c_size_t
        ci = ctypes.c_int
        L.cmpq_collect_stats.argtypes = [vp, ci, i64, i64, i64, vp, vp, vp, sz, vp]
        L.cmpq_check_finite.argtypes = [vp, vp]
        L.cmpq_check_finite.restype = ci
        L.cmpq_collect_stats_static.argtypes = [vp, ci, i64, i64, i64, vp, vp]
        L.cmpq_finalize_stats.argtypes = [vp, i64, vp, vp]
        L.cmpq_allocate_bits.argtypes = [vp, i64, dbl, ci, vp, vp, vp, sz, vp]
        L.cmpq_extract_outliers.argtypes = [vp, ci, i64, i64, i64, vp, vp, i64, i64, ci, vp, vp, vp,
                                            i64, vp, vp, sz, vp]
        L.cmpq_quantize_layer.argtypes = [vp, ci, i64, i64, i64, vp, vp, vp, i64, ci, vp, vp, vp, vp,
                                          vp, vp, vp, sz, vp]
        L.cmpq_pack.argtypes = [vp, vp, i64, i64, vp, vp, vp, vp, vp, sz, vp]
        L.cmpq_protect_and_quantize.argtypes = [vp, ci, i64, i64, i64, vp, vp, i64, i64, ci, vp, vp, vp, i64, vp,
                                                vp, vp, vp, vp, vp, sz, vp]
        L.cmpq_protect_and_quantize.restype = ci
        L.cmpq_collect_stats_norm.argtypes = [vp, ci, i64, i64, i64, ci, vp, vp, vp, sz, vp]
        L.cmpq_collect_stats_norm.restype = ci
        L.cmpq_finalize_stats_norm.argtypes = [vp, i64, ci, vp, vp]
        L.cmpq_finalize_stats_norm.restype = ci
        L.cmpq_transpose16.argtypes = [vp, i64, i64, i64, vp, i64, vp]
        L.cmpq_transpose16.restype = ci
        L.cmpq_matvec.argtypes = [vp, vp, vp, vp, vp, i64, i64, vp, ci, vp, vp, vp, vp, vp, vp, sz, vp]
        L.cmpq_matvec.restype = ci
        L.cmpq_outliers_by_column.argtypes = [vp, vp, vp, i64, i64, vp, vp, vp, vp, sz, vp]
        L.cmpq_outliers_by_column.restype = ci
        for name in ("cmpq_collect_stats", "cmpq_collect_stats_static", "cmpq_finalize_stats", "cmpq_allocate_bits",
                     "cmpq_extract_outliers", "cmpq_quantize_layer", "cmpq_pack"):
            getattr(L, name).restype = ci
        L.cmpq_workspace_bytes.argtypes = [ci, i64, i64]
        L.cmpq_workspace_bytes.restype = sz
        L.cmpq_alloc_counts.argtypes = [i64, dbl, ctypes.POINTER(i64), ctypes.POINTER(i64)]
        L.cmpq_alloc_counts.restype = None
        L.cmpq_default_counts.argtypes = [i64, i64, ctypes.POINTER(i64), ctypes.POINTER(i64)]
        L.cmpq_default_counts.restype = None
        L.cmpq_packed_words.argtypes = [vp, i64, i64]
        L.cmpq_packed_words.restype = i64
        L.cmpq_set_lloyd_assignment.argtypes = [ci]
        L.cmpq_set_lloyd_assignment.restype = ci
        L.cmpq_get_lloyd_assignment.argtypes = []
        L.cmpq_get_lloyd_assignment.restype = ci
        L.cmpq_lloyd_phase_events.argtypes = [vp, vp, vp, vp]
        L.cmpq_lloyd_phase_events.restype = ci
        L.cmpq_sweep_cache_bytes.argtypes = [i64, i64]
        L.cmpq_sweep_cache_bytes.restype = sz
        L.cmpq_sweep_begin.argtypes = [vp, ci, i64, i64, i64, ci, vp, vp, sz, vp]
        L.cmpq_sweep_begin.restype = ci
        L.cmpq_sweep_budget.argtypes = [vp, ci, i64, i64, i64, vp, vp, i64, i64, ci, vp, vp, vp, i64, vp,
                                        vp, vp, vp, vp, sz, vp, sz, vp]
        L.cmpq_sweep_budget.restype = ci
        L.cmpq_sweep_budget_pack.argtypes = [vp, ci, i64, i64, i64, vp, vp, i64, i64, ci, vp, vp, vp, i64, vp,
                                             vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, sz, vp]
        L.cmpq_sweep_budget_pack.restype = ci
        L.cmpq_quantize_layer_packed.argtypes = [vp, ci, i64, i64, i64, vp, vp, vp, i64, ci, vp, vp, vp, vp, vp, vp,
                                                 vp, vp, vp, vp, vp, sz, vp]
        L.cmpq_quantize_layer_packed.restype = ci
        L.cmpq_protect_quantize_pack.argtypes = [vp, ci, i64, i64, i64, vp, vp, i64, i64, ci, vp, vp, vp, i64, vp,
                                                 vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.cmpq_protect_quantize_pack.restype = ci
        L.cmpq_matvec_f16lut.argtypes = L.cmpq_matvec.argtypes
        L.cmpq_matvec_f16lut.restype = ci
        L.cmpq_lut_bytes.argtypes = [ci, i64]
        L.cmpq_lut_bytes.restype = sz
        L.cmpq_store_lut.argtypes = [vp, vp, i64, ci, vp, vp]
        L.cmpq_store_lut.restype = ci
        L.cmpq_load_lut.argtypes = [vp, ci, vp, i64, vp, vp]
        L.cmpq_load_lut.restype = ci
        L.cmpq_table_bits_per_weight.argtypes = [vp, i64, i64, ci, ci]
        L.cmpq_table_bits_per_weight.restype = dbl
        L.cmpq_alu_probe.argtypes = [ci, ci, vp, ctypes.POINTER(ctypes.c_ulonglong), vp]
        L.cmpq_alu_probe.restype = ci
        L.cmpq_kernel_resources.argtypes = [ci, ctypes.POINTER(ci), ctypes.POINTER(ci)]
        L.cmpq_kernel_resources.restype = ci
        L.cmpq_status_string.argtypes = [ci]
        L.cmpq_status_string.restype = ctypes.c_char_p
        _lib = L
    return _lib


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status, where):
    if status != 0:
        raise CmpqError(status, where)


def dtype_code(t):
    if t.dtype == torch.float16:
        return F16
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("expected a float16 or bfloat16 tensor, got %s" % t.dtype)


def cmpq_workspace_bytes(op, d_in, d_out=0):
    return int(lib().cmpq_workspace_bytes(op, d_in, d_out))


def workspace(op, d_in, d_out=0, device="cuda"):
    """A fresh scratch buffer of the size the given call needs."""
    return torch.empty(max(256, cmpq_workspace_bytes(op, d_in, d_out)), dtype=torch.uint8, device=device)


def cmpq_set_lloyd_assignment(mode):
    """ASSIGN_ORDERED (default) or ASSIGN_ALL_PAIRS for the K-means calls that follow."""
    _check(lib().cmpq_set_lloyd_assignment(int(mode)), "cmpq_set_lloyd_assignment")


def cmpq_get_lloyd_assignment():
    return int(lib().cmpq_get_lloyd_assignment())


def cmpq_lloyd_phase_events(events):
    """`events`: four torch.cuda.Event(enable_timing=True) that the next ordered K-means call records
    before its table kernel and after its table, iterate and assign kernels; None cancels."""
    if events is None:
        _check(lib().cmpq_lloyd_phase_events(None, None, None, None), "cmpq_lloyd_phase_events")
        return
    handles = []
    for ev in events:
        ev.record()  # torch creates the CUDA event lazily: make sure the handle exists
        handles.append(ctypes.c_void_p(ev.cuda_event))
    _check(lib().cmpq_lloyd_phase_events(*handles), "cmpq_lloyd_phase_events")


KERNEL_STATS_PARTIAL_VEC_BF16, KERNEL_LLOYD_TABLE_BF16_4096 = 0, 1


def cmpq_alu_probe(rounds, blocks, sink):
    """Enqueues the arithmetic-throughput probe; returns the (value, centroid) pairs it evaluates."""
    n = ctypes.c_ulonglong()
    _check(lib().cmpq_alu_probe(int(rounds), int(blocks), _ptr(sink), ctypes.byref(n), _stream()), "cmpq_alu_probe")
    return int(n.value)


def cmpq_kernel_resources(kernel):
    """(registers per thread, static shared memory bytes) of one of the library's kernels as compiled."""
    regs, smem = ctypes.c_int(), ctypes.c_int()
    _check(lib().cmpq_kernel_resources(int(kernel), ctypes.byref(regs), ctypes.byref(smem)), "cmpq_kernel_resources")
    return regs.value, smem.value


def cmpq_alloc_counts(d_in, avg_bits):
    n2, n4 = ctypes.c_int64(), ctypes.c_int64()
    lib().cmpq_alloc_counts(d_in, avg_bits, ctypes.byref(n2), ctypes.byref(n4))
    return n2.value, n4.value


def cmpq_default_counts(d_in, d_out):
    n_act, n_q = ctypes.c_int64(), ctypes.c_int64()
    lib().cmpq_default_counts(d_in, d_out, ctypes.byref(n_act), ctypes.byref(n_q))
    return n_act.value, n_q.value


def cmpq_packed_words(bits_host, d_out):
    """bits_host: a CPU uint8 tensor."""
    b = bits_host.contiguous()
    return int(lib().cmpq_packed_words(ctypes.c_void_p(b.data_ptr()), b.numel(), d_out))


def cmpq_collect_stats(X, sumsq, ws, nonfinite=None):
    """sumsq (float64 [d_in]) += column sums of squares of X ([n_tokens][d_in], fp16/bf16).
    nonfinite (here and below): optional int32 device word the kernels OR their findings into
    (bit 0: a NaN or infinity among the activations, bit 1: among the weights); see cmpq_check_finite."""
    n, d_in = X.shape
    _check(lib().cmpq_collect_stats(_ptr(X), dtype_code(X), n, d_in, X.stride(0) if n > 0 else d_in,
                                    _ptr(sumsq), _ptr(nonfinite), _ptr(ws), ws.numel(), _stream()), "cmpq_collect_stats")


def cmpq_check_finite(nonfinite):
    """Waits for the current stream; raises CmpqError (status 6) if the word is not zero."""
    _check(lib().cmpq_check_finite(_ptr(nonfinite), _stream()), "cmpq_check_finite")


def cmpq_collect_stats_static(X, sumsq):
    """cmpq_collect_stats for callers that cannot provide a work space: the scratch is a fixed array
    inside the library (d_in <= 32768).  Calls on different streams must not overlap."""
    n, d_in = X.shape
    _check(lib().cmpq_collect_stats_static(_ptr(X), dtype_code(X), n, d_in, X.stride(0) if n > 0 else d_in,
                                           _ptr(sumsq), _stream()), "cmpq_collect_stats_static")


def cmpq_finalize_stats(sumsq, a):
    _check(lib().cmpq_finalize_stats(_ptr(sumsq), sumsq.numel(), _ptr(a), _stream()), "cmpq_finalize_stats")


def cmpq_allocate_bits(a, avg_bits, mode, bits, order, ws):
    _check(lib().cmpq_allocate_bits(_ptr(a), a.numel(), float(avg_bits), int(mode), _ptr(bits), _ptr(order),
                                    _ptr(ws), ws.numel(), _stream()), "cmpq_allocate_bits")


def cmpq_extract_outliers(W, a, bits, n_act, n_q, lloyd_iters, rows, cols, vals, ws, nonfinite=None):
    d_in, d_out = W.shape
    _check(lib().cmpq_extract_outliers(_ptr(W), dtype_code(W), d_in, d_out, W.stride(0), _ptr(a), _ptr(bits),
                                       n_act, n_q, lloyd_iters, _ptr(rows), _ptr(cols), _ptr(vals),
                                       rows.numel(), _ptr(nonfinite), _ptr(ws), ws.numel(), _stream()),
           "cmpq_extract_outliers")


def cmpq_quantize_layer(W, bits, rows, cols, lloyd_iters, lut, codes, ws, sens=None, inexact_rows=None,
                        sweeps=None, nonfinite=None):
    d_in, d_out = W.shape
    nnz = 0 if rows is None else rows.numel()
    _check(lib().cmpq_quantize_layer(_ptr(W), dtype_code(W), d_in, d_out, W.stride(0), _ptr(bits),
                                     _ptr(rows) if nnz else None, _ptr(cols) if nnz else None, nnz,
                                     lloyd_iters, _ptr(sens), _ptr(lut), _ptr(codes), _ptr(inexact_rows),
                                     _ptr(sweeps), _ptr(nonfinite), _ptr(ws), ws.numel(), _stream()),
           "cmpq_quantize_layer")


def cmpq_protect_and_quantize(W, a, bits, n_act, n_q, lloyd_iters, rows, cols, vals, lut, codes, ws,
                              inexact_rows=None, sweeps=None, nonfinite=None):
    d_in, d_out = W.shape
    nnz = n_act * d_out + n_q
    _check(lib().cmpq_protect_and_quantize(_ptr(W), dtype_code(W), d_in, d_out, W.stride(0), _ptr(a), _ptr(bits),
                                           n_act, n_q, lloyd_iters, _ptr(rows), _ptr(cols), _ptr(vals), nnz,
                                           _ptr(lut), _ptr(codes), _ptr(inexact_rows), _ptr(sweeps), _ptr(nonfinite),
                                           _ptr(ws), ws.numel(), _stream()), "cmpq_protect_and_quantize")


def cmpq_quantize_layer_packed(W, bits, rows, cols, lloyd_iters, lut, codes, packed, row_off, perm, seg_rows, ws,
                               sens=None, inexact_rows=None, sweeps=None, nonfinite=None):
    """cmpq_quantize_layer and cmpq_pack in one call; codes may be None (the byte codes are then never written)."""
    d_in, d_out = W.shape
    nnz = 0 if rows is None else rows.numel()
    _check(lib().cmpq_quantize_layer_packed(_ptr(W), dtype_code(W), d_in, d_out, W.stride(0), _ptr(bits),
                                            _ptr(rows) if nnz else None, _ptr(cols) if nnz else None, nnz,
                                            lloyd_iters, _ptr(sens), _ptr(lut), _ptr(codes), _ptr(packed),
                                            _ptr(row_off), _ptr(perm), _ptr(seg_rows), _ptr(inexact_rows),
                                            _ptr(sweeps), _ptr(nonfinite), _ptr(ws), ws.numel(), _stream()),
           "cmpq_quantize_layer_packed")


def cmpq_protect_quantize_pack(W, a, bits, n_act, n_q, lloyd_iters, rows, cols, vals, lut, codes, packed, row_off,
                               perm, seg_rows, ws, inexact_rows=None, sweeps=None, nonfinite=None):
    """cmpq_protect_and_quantize and cmpq_pack in one call; codes may be None."""
    d_in, d_out = W.shape
    nnz = n_act * d_out + n_q
    _check(lib().cmpq_protect_quantize_pack(_ptr(W), dtype_code(W), d_in, d_out, W.stride(0), _ptr(a), _ptr(bits),
                                            n_act, n_q, lloyd_iters, _ptr(rows), _ptr(cols), _ptr(vals), nnz,
                                            _ptr(lut), _ptr(codes), _ptr(packed), _ptr(row_off), _ptr(perm),
                                            _ptr(seg_rows), _ptr(inexact_rows), _ptr(sweeps), _ptr(nonfinite),
                                            _ptr(ws), ws.numel(), _stream()), "cmpq_protect_quantize_pack")


def cmpq_sweep_cache_bytes(d_in, d_out):
    return int(lib().cmpq_sweep_cache_bytes(d_in, d_out))


def cmpq_sweep_begin(W, lloyd_iters, cache, nonfinite=None):
    """Counts the values of every channel of W into `cache` (uint8 tensor of cmpq_sweep_cache_bytes bytes)."""
    d_in, d_out = W.shape
    _check(lib().cmpq_sweep_begin(_ptr(W), dtype_code(W), d_in, d_out, W.stride(0), lloyd_iters, _ptr(nonfinite),
                                  _ptr(cache), cache.numel(), _stream()), "cmpq_sweep_begin")


def cmpq_sweep_budget(W, a, bits, n_act, n_q, lloyd_iters, rows, cols, vals, lut, codes, cache, ws,
                      inexact_rows=None, sweeps=None):
    """cmpq_protect_and_quantize with the value tables and provisional fits kept in `cache`."""
    d_in, d_out = W.shape
    nnz = n_act * d_out + n_q
    _check(lib().cmpq_sweep_budget(_ptr(W), dtype_code(W), d_in, d_out, W.stride(0), _ptr(a), _ptr(bits),
                                   n_act, n_q, lloyd_iters, _ptr(rows), _ptr(cols), _ptr(vals), nnz, _ptr(lut),
                                   _ptr(codes), _ptr(inexact_rows), _ptr(sweeps), _ptr(cache), cache.numel(),
                                   _ptr(ws), ws.numel(), _stream()), "cmpq_sweep_budget")


def cmpq_sweep_budget_pack(W, a, bits, n_act, n_q, lloyd_iters, rows, cols, vals, lut, codes, packed, row_off, perm,
                           seg_rows, cache, ws, inexact_rows=None, sweeps=None):
    """cmpq_protect_quantize_pack with the value tables and provisional fits kept in `cache`; codes may be None."""
    d_in, d_out = W.shape
    nnz = n_act * d_out + n_q
    _check(lib().cmpq_sweep_budget_pack(_ptr(W), dtype_code(W), d_in, d_out, W.stride(0), _ptr(a), _ptr(bits),
                                        n_act, n_q, lloyd_iters, _ptr(rows), _ptr(cols), _ptr(vals), nnz, _ptr(lut),
                                        _ptr(codes), _ptr(packed), _ptr(row_off), _ptr(perm), _ptr(seg_rows),
                                        _ptr(inexact_rows), _ptr(sweeps), _ptr(cache), cache.numel(), _ptr(ws),
                                        ws.numel(), _stream()), "cmpq_sweep_budget_pack")


def cmpq_pack(codes, bits, packed, row_off, perm, seg_rows, ws):
    d_in, d_out = codes.shape
    _check(lib().cmpq_pack(_ptr(codes), _ptr(bits), d_in, d_out, _ptr(packed), _ptr(row_off), _ptr(perm),
                           _ptr(seg_rows), _ptr(ws), ws.numel(), _stream()), "cmpq_pack")


def cmpq_outliers_by_column(rows, cols, vals, d_out, col_ptr, c_rows, c_vals, ws):
    """Regroups the (row, col)-sorted outlier list by column: col_ptr int64 [d_out+1], c_rows int32 [nnz],
    c_vals 16-bit patterns [nnz]."""
    nnz = 0 if rows is None else rows.numel()
    _check(lib().cmpq_outliers_by_column(_ptr(rows) if nnz else None, _ptr(cols) if nnz else None,
                                         _ptr(vals) if nnz else None, nnz, d_out, _ptr(col_ptr),
                                         _ptr(c_rows) if nnz else None, _ptr(c_vals) if nnz else None,
                                         _ptr(ws), ws.numel(), _stream()), "cmpq_outliers_by_column")


def cmpq_matvec(packed, row_off, perm, seg_rows, lut, x, col_ptr, c_rows, c_vals, y, y16, ws):
    """y (float32 [d_out]) = x (fp16/bf16 [d_in]) times the quantized layer read from its packed segments,
    plus the outlier products; y16 (optional) receives y rounded to x's dtype."""
    d_in, d_out = x.numel(), y.numel()
    _check(lib().cmpq_matvec(_ptr(packed), _ptr(row_off), _ptr(perm), _ptr(seg_rows), _ptr(lut), d_in, d_out,
                             _ptr(x), dtype_code(x), _ptr(col_ptr), _ptr(c_rows), _ptr(c_vals), _ptr(y),
                             _ptr(y16), _ptr(ws), ws.numel(), _stream()), "cmpq_matvec")


LUT_F32, LUT_F16, LUT_U4 = 0, 1, 2
LUT_U4_BYTES = 12


def cmpq_lut_bytes(fmt, d_in):
    return int(lib().cmpq_lut_bytes(int(fmt), d_in))


def cmpq_store_lut(lut, bits, fmt, stored):
    """lut (float32 [d_in][16]) -> stored: int16 [d_in][16] (LUT_F16) or uint8 [d_in][12] (LUT_U4)."""
    _check(lib().cmpq_store_lut(_ptr(lut), _ptr(bits), lut.shape[0], int(fmt), _ptr(stored), _stream()),
           "cmpq_store_lut")


def cmpq_load_lut(stored, fmt, bits, lut):
    _check(lib().cmpq_load_lut(_ptr(stored), int(fmt), _ptr(bits), lut.shape[0], _ptr(lut), _stream()),
           "cmpq_load_lut")


def cmpq_table_bits_per_weight(bits_host, d_out, fmt, count_grid_ends=False):
    """bits_host: a CPU uint8 tensor.  The table and width-tag overhead in bits per weight."""
    b = bits_host.contiguous()
    return float(lib().cmpq_table_bits_per_weight(ctypes.c_void_p(b.data_ptr()), b.numel(), d_out, int(fmt),
                                                  1 if count_grid_ends else 0))


def cmpq_matvec_f16lut(packed, row_off, perm, seg_rows, lut16, x, col_ptr, c_rows, c_vals, y, y16, ws):
    """cmpq_matvec reading the tables in their stored FP16 format (int16 [d_in][16])."""
    d_in, d_out = x.numel(), y.numel()
    _check(lib().cmpq_matvec_f16lut(_ptr(packed), _ptr(row_off), _ptr(perm), _ptr(seg_rows), _ptr(lut16), d_in,
                                    d_out, _ptr(x), dtype_code(x), _ptr(col_ptr), _ptr(c_rows), _ptr(c_vals),
                                    _ptr(y), _ptr(y16), _ptr(ws), ws.numel(), _stream()), "cmpq_matvec_f16lut")


def cmpq_collect_stats_norm(X, norm, acc, ws, nonfinite=None):
    """acc (float64 [d_in]) accumulates the l2 / l1 / l_inf statistic of X's columns (NORM_L2, NORM_L1, NORM_LINF)."""
    n, d_in = X.shape
    _check(lib().cmpq_collect_stats_norm(_ptr(X), dtype_code(X), n, d_in, X.stride(0) if n > 0 else d_in, int(norm),
                                         _ptr(acc), _ptr(nonfinite), _ptr(ws), ws.numel(), _stream()),
           "cmpq_collect_stats_norm")


def cmpq_finalize_stats_norm(acc, norm, a):
    _check(lib().cmpq_finalize_stats_norm(_ptr(acc), acc.numel(), int(norm), _ptr(a), _stream()),
           "cmpq_finalize_stats_norm")


def cmpq_transpose16(src, dst):
    """dst[c][r] = src[r][c] for 2-D fp16/bf16 tensors with unit inner stride (e.g. a framework's [d_out][d_in]
    weight into the [d_in][d_out] layout the other calls take)."""
    rows, cols = src.shape
    if src.stride(1) != 1 or dst.stride(1) != 1 or tuple(dst.shape) != (cols, rows) or src.dtype != dst.dtype:
        raise ValueError("cmpq_transpose16 needs row-major 2-D tensors of one dtype with shapes [r][c] and [c][r]")
    dtype_code(src)
    _check(lib().cmpq_transpose16(_ptr(src), rows, cols, src.stride(0), _ptr(dst), dst.stride(0), _stream()),
           "cmpq_transpose16")
