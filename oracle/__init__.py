"""CMPQ oracle: ctypes binding of ``cmpq_oracle.c`` -- TEST INFRASTRUCTURE ONLY.

A plain single-threaded CPU restatement of the CMPQ pass (arxiv 2410.13056,
Sections 3.2.1 and 3.2.2, Algorithm 1, Section 5.1).  Only the tests, the smoke
check and the benchmark's CPU-baseline leg may import this package; the CUDA
library never does, and this package never imports the CUDA library.

All arrays are numpy arrays; 16-bit float tensors travel as ``uint16`` bit
patterns together with ``dtype`` (0 = fp16, 1 = bf16).
"""
import ctypes
import os
import subprocess

import numpy as np

F16 = 0
BF16 = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cmpq_oracle.c")
_LIB_PATH = os.path.join(_HERE, "libcmpq_oracle.so")
_lib = None


def build(force=False):
    """Compile the oracle with gcc (-O2, no contraction, no fast-math)."""
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= os.path.getmtime(_SRC)):
        return _LIB_PATH
    tmp = _LIB_PATH + ".tmp%d" % os.getpid()
    subprocess.run(["gcc", "-O2", "-ffp-contract=off", "-std=c11", "-Wall", "-shared", "-fPIC",
                    "-o", tmp, _SRC, "-lm"], check=True)
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_widen.restype = ctypes.c_float
        _lib.oracle_widen.argtypes = [ctypes.c_uint16, ctypes.c_int]
        _lib.oracle_packed_words.restype = ctypes.c_int64
        _lib.oracle_metadata_bits_per_weight.restype = ctypes.c_double
        _lib.oracle_recon_error.restype = ctypes.c_double
        _lib.oracle_float_to_half.restype = ctypes.c_uint16
        _lib.oracle_float_to_half.argtypes = [ctypes.c_float]
    return _lib


def _p(arr):
    return None if arr is None else arr.ctypes.data_as(ctypes.c_void_p)


def _i64(v):
    return ctypes.c_int64(int(v))


def _c(arr, dt):
    arr = np.ascontiguousarray(arr, dtype=dt)
    return arr


def widen(u16, dtype):
    """Exact fp16/bf16 bit pattern -> float32 (element by element through the C routine)."""
    u16 = _c(u16, np.uint16)
    out = np.empty(u16.shape, np.float32)
    flat_in, flat_out = u16.reshape(-1), out.reshape(-1)
    f = lib().oracle_widen
    for i in range(flat_in.size):
        flat_out[i] = f(int(flat_in[i]), dtype)
    return out


def collect_stats(X_u16, dtype, sumsq=None):
    X_u16 = _c(X_u16, np.uint16)
    n, d_in = X_u16.shape
    if sumsq is None:
        sumsq = np.zeros(d_in, np.float64)
    lib().oracle_collect_stats(_p(X_u16), dtype, _i64(n), _i64(d_in), _i64(d_in), _p(sumsq))
    return sumsq


def finalize_stats(sumsq):
    sumsq = _c(sumsq, np.float64)
    a = np.empty(sumsq.shape[0], np.float32)
    lib().oracle_finalize_stats(_p(sumsq), _i64(sumsq.shape[0]), _p(a))
    return a


NORM_L2, NORM_L1, NORM_LINF = 0, 1, 2


def collect_stats_norm(X_u16, dtype, norm, acc=None):
    """Accumulates the l2 (sum of squares), l1 (sum of magnitudes) or l_inf (largest magnitude) statistic."""
    X_u16 = _c(X_u16, np.uint16)
    n, d_in = X_u16.shape
    if acc is None:
        acc = np.zeros(d_in, np.float64)
    lib().oracle_collect_stats_norm(_p(X_u16), dtype, _i64(n), _i64(d_in), _i64(d_in), int(norm), _p(acc))
    return acc


def finalize_stats_norm(acc, norm):
    acc = _c(acc, np.float64)
    a = np.empty(acc.shape[0], np.float32)
    lib().oracle_finalize_stats_norm(_p(acc), _i64(acc.shape[0]), int(norm), _p(a))
    return a


def alloc_counts(d_in, avg_bits):
    n2, n4 = ctypes.c_int64(), ctypes.c_int64()
    lib().oracle_alloc_counts(_i64(d_in), ctypes.c_double(avg_bits), ctypes.byref(n2),
                              ctypes.byref(n4))
    return n2.value, n4.value


def default_counts(d_in, d_out):
    n_act, n_q = ctypes.c_int64(), ctypes.c_int64()
    lib().oracle_default_counts(_i64(d_in), _i64(d_out), ctypes.byref(n_act), ctypes.byref(n_q))
    return n_act.value, n_q.value


def allocate_bits(a, avg_bits, mode=0):
    """Algorithm 1.  Returns (bits uint8[d_in], order int32[d_in])."""
    a = _c(a, np.float32)
    d_in = a.shape[0]
    bits = np.empty(d_in, np.uint8)
    order = np.empty(d_in, np.int32)
    rc = lib().oracle_allocate_bits(_p(a), _i64(d_in), ctypes.c_double(avg_bits), int(mode),
                                    _p(bits), _p(order))
    if rc:
        raise ValueError("avg_bits must lie in [2, 4]")
    return bits, order


def lloyd(x, K, T, s=None, trace=False):
    """Channel K-means.  Returns (lut float32[16], code uint8[N], err float32[N][, sse[T+1]])."""
    x = _c(x, np.float32)
    N = x.shape[0]
    lut = np.zeros(16, np.float32)
    code = np.empty(N, np.uint8)
    err = np.empty(N, np.float32)
    sse = np.zeros(T + 1, np.float64) if trace else None
    if s is not None:
        s = _c(s, np.float64)
    lib().oracle_lloyd(_p(x), _i64(N), int(K), int(T), _p(s), _p(lut), _p(code), _p(err), _p(sse))
    return (lut, code, err, sse) if trace else (lut, code, err)


def extract_outliers(W_u16, dtype, a, bits, n_act, n_q, T, want_fit=False):
    """Section 3.2.2.  Returns (rows, cols, vals[, lut1, err])."""
    W_u16 = _c(W_u16, np.uint16)
    d_in, d_out = W_u16.shape
    a = _c(a, np.float32)
    bits = _c(bits, np.uint8)
    nnz = n_act * d_out + n_q
    rows = np.empty(nnz, np.int32)
    cols = np.empty(nnz, np.int32)
    vals = np.empty(nnz, np.uint16)
    lut1 = np.zeros((d_in, 16), np.float32) if want_fit else None
    err = np.zeros((d_in, d_out), np.float32) if want_fit else None
    rc = lib().oracle_extract_outliers(_p(W_u16), dtype, _i64(d_in), _i64(d_out), _i64(d_out),
                                       _p(a), _p(bits), _i64(n_act), _i64(n_q), int(T),
                                       _p(rows), _p(cols), _p(vals), _p(lut1), _p(err))
    if rc:
        raise ValueError("bad outlier counts")
    return (rows, cols, vals, lut1, err) if want_fit else (rows, cols, vals)


def quantize_layer(W_u16, dtype, bits, rows, cols, T, sens=None):
    """Final channel-wise K-means on W - O.  Returns (lut float32[d_in,16], codes uint8[d_in,d_out])."""
    W_u16 = _c(W_u16, np.uint16)
    d_in, d_out = W_u16.shape
    bits = _c(bits, np.uint8)
    rows = _c(rows, np.int32)
    cols = _c(cols, np.int32)
    lut = np.zeros((d_in, 16), np.float32)
    codes = np.empty((d_in, d_out), np.uint8)
    if sens is not None:
        sens = _c(sens, np.float64)
    rc = lib().oracle_quantize_layer(_p(W_u16), dtype, _i64(d_in), _i64(d_out), _i64(d_out),
                                     _p(bits), _p(rows), _p(cols), _i64(rows.shape[0]), int(T),
                                     _p(sens), _p(lut), _p(codes))
    if rc:
        raise ValueError("outlier rows must be sorted ascending")
    return lut, codes


def packed_words(bits, d_out):
    bits = _c(bits, np.uint8)
    return int(lib().oracle_packed_words(_p(bits), _i64(bits.shape[0]), _i64(d_out)))


def pack(codes, bits):
    """Returns (packed uint32[words], row_off int64[d_in+1], perm int32[d_in], seg_rows int64[3])."""
    codes = _c(codes, np.uint8)
    bits = _c(bits, np.uint8)
    d_in, d_out = codes.shape
    packed = np.empty(packed_words(bits, d_out), np.uint32)
    row_off = np.empty(d_in + 1, np.int64)
    perm = np.empty(d_in, np.int32)
    seg_rows = np.zeros(3, np.int64)
    lib().oracle_pack(_p(codes), _p(bits), _i64(d_in), _i64(d_out), _p(packed), _p(row_off),
                      _p(perm), _p(seg_rows))
    return packed, row_off, perm, seg_rows


def unpack(packed, row_off, perm, bits, d_out):
    packed = _c(packed, np.uint32)
    row_off = _c(row_off, np.int64)
    perm = _c(perm, np.int32)
    bits = _c(bits, np.uint8)
    d_in = bits.shape[0]
    codes = np.empty((d_in, d_out), np.uint8)
    lib().oracle_unpack(_p(packed), _p(row_off), _p(perm), _p(bits), _i64(d_in), _i64(d_out),
                        _p(codes))
    return codes


def metadata_bits_per_weight(bits, d_out, tag_bits=4, lut_bits=16):
    bits = _c(bits, np.uint8)
    return float(lib().oracle_metadata_bits_per_weight(_p(bits), _i64(bits.shape[0]), _i64(d_out),
                                                       int(tag_bits), int(lut_bits)))


def float_to_half(values):
    """float32 -> binary16 bit patterns, round to nearest even (element by element through the C routine)."""
    v = _c(values, np.float32).reshape(-1)
    f = lib().oracle_float_to_half
    return np.array([f(ctypes.c_float(float(x))) for x in v], np.uint16).reshape(np.shape(values))


LUT_U4_BYTES = 12


def lut_to_f16(lut, bits):
    """Tables rounded to FP16 (Section 5.1): uint16 [d_in][16], entries beyond K are 0."""
    lut = _c(lut, np.float32)
    bits = _c(bits, np.uint8)
    out = np.empty((bits.shape[0], 16), np.uint16)
    lib().oracle_lut_to_f16(_p(lut), _p(bits), _i64(bits.shape[0]), _p(out))
    return out


def lut_from_f16(lut16):
    lut16 = _c(lut16, np.uint16)
    out = np.empty(lut16.shape, np.float32)
    lib().oracle_lut_from_f16(_p(lut16), _i64(lut16.shape[0]), _p(out))
    return out


def lut_to_u4(lut, bits):
    """Tables in 4 bits per centroid (Section 5.1 variant): uint8 [d_in][12] = 8 code bytes + FP16 lo, hi."""
    lut = _c(lut, np.float32)
    bits = _c(bits, np.uint8)
    out = np.empty((bits.shape[0], LUT_U4_BYTES), np.uint8)
    lib().oracle_lut_to_u4(_p(lut), _p(bits), _i64(bits.shape[0]), _p(out))
    return out


def lut_from_u4(stored, bits):
    stored = _c(stored, np.uint8)
    bits = _c(bits, np.uint8)
    out = np.empty((bits.shape[0], 16), np.float32)
    lib().oracle_lut_from_u4(_p(stored), _p(bits), _i64(bits.shape[0]), _p(out))
    return out


def recon_error(X_u16, W_u16, dtype, lut, codes, rows, cols, vals, t_step=1):
    """E = ||X (W - What)||_F in fp64, What = lut[code] + O (every t_step-th token)."""
    X_u16 = _c(X_u16, np.uint16)
    W_u16 = _c(W_u16, np.uint16)
    n, d_in = X_u16.shape
    d_out = W_u16.shape[1]
    lut = _c(lut, np.float32)
    codes = _c(codes, np.uint8)
    rows = _c(rows, np.int32)
    cols = _c(cols, np.int32)
    vals = _c(vals, np.uint16)
    return float(lib().oracle_recon_error(_p(X_u16), _p(W_u16), dtype, _i64(n), _i64(d_in),
                                          _i64(d_out), _i64(d_in), _i64(d_out), _p(lut), _p(codes),
                                          _p(rows), _p(cols), _p(vals), _i64(rows.shape[0]),
                                          _i64(t_step)))


def matvec(x_u16, dtype, lut, codes, rows, cols, vals):
    """Inference product of one token (Section 6): returns (y float64[d_out], yabs float64[d_out])."""
    x_u16 = _c(x_u16, np.uint16)
    lut = _c(lut, np.float32)
    codes = _c(codes, np.uint8)
    rows = _c(rows, np.int32)
    cols = _c(cols, np.int32)
    vals = _c(vals, np.uint16)
    d_in, d_out = codes.shape
    y = np.empty(d_out, np.float64)
    yabs = np.empty(d_out, np.float64)
    lib().oracle_matvec(_p(x_u16), dtype, _i64(d_in), _i64(d_out), _p(lut), _p(codes), _p(rows),
                        _p(cols), _p(vals), _i64(rows.shape[0]), _p(y), _p(yabs))
    return y, yabs


def outliers_by_column(rows, cols, vals, d_out):
    """Outlier list regrouped by column.  Returns (col_ptr int64[d_out+1], rows int32, vals uint16)."""
    rows = _c(rows, np.int32)
    cols = _c(cols, np.int32)
    vals = _c(vals, np.uint16)
    nnz = rows.shape[0]
    col_ptr = np.empty(d_out + 1, np.int64)
    c_rows = np.empty(nnz, np.int32)
    c_vals = np.empty(nnz, np.uint16)
    lib().oracle_outliers_by_column(_p(rows), _p(cols), _p(vals), _i64(nnz), _i64(d_out),
                                    _p(col_ptr), _p(c_rows), _p(c_vals))
    return col_ptr, c_rows, c_vals


def layer_pass(X_u16, W_u16, dtype, avg_bits, n_act, n_q, T):
    """The whole pass for one layer in the paper's order; returns a dict of all outputs."""
    X_u16 = _c(X_u16, np.uint16)
    W_u16 = _c(W_u16, np.uint16)
    n, d_in = X_u16.shape
    d_out = W_u16.shape[1]
    nnz = n_act * d_out + n_q
    out = dict(a=np.empty(d_in, np.float32), bits=np.empty(d_in, np.uint8),
               rows=np.empty(nnz, np.int32), cols=np.empty(nnz, np.int32),
               vals=np.empty(nnz, np.uint16), lut=np.zeros((d_in, 16), np.float32),
               codes=np.empty((d_in, d_out), np.uint8),
               packed=np.zeros(d_in * ((d_out * 4 + 31) // 32), np.uint32),
               row_off=np.empty(d_in + 1, np.int64), perm=np.empty(d_in, np.int32),
               seg_rows=np.zeros(3, np.int64))
    rc = lib().oracle_layer_pass(_p(X_u16), _p(W_u16), dtype, _i64(n), _i64(d_in), _i64(d_out),
                                 _i64(d_in), _i64(d_out), ctypes.c_double(avg_bits), _i64(n_act),
                                 _i64(n_q), int(T), _p(out["a"]), _p(out["bits"]), _p(out["rows"]),
                                 _p(out["cols"]), _p(out["vals"]), _p(out["lut"]), _p(out["codes"]),
                                 _p(out["packed"]), _p(out["row_off"]), _p(out["perm"]),
                                 _p(out["seg_rows"]))
    if rc:
        raise ValueError("oracle_layer_pass failed with %d" % rc)
    out["packed"] = out["packed"][: int(out["row_off"][-1])]
    return out
