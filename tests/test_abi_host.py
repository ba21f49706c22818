"""Host-side checks of the C ABI that need no GPU: the library loads, exports what the header
declares, its pure helpers agree with the checker, and bad arguments are refused before any
launch."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2410_13056_b200 import binding as B
from paper_2410_13056_b200 import build as cuda_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    cuda_build.build()
    return B.lib()


def test_every_declared_symbol_is_exported(L):
    header = open(os.path.join(ROOT, "include", "cmpq.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(cmpq_[a-z0-9_]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


def test_status_strings(L):
    assert L.cmpq_status_string(0) == b"ok"
    assert len({L.cmpq_status_string(s) for s in range(6)}) == 6


@pytest.mark.parametrize("d_in", [1, 7, 512, 4096, 11008, 28672])
@pytest.mark.parametrize("b", [2.0, 2.2, 2.5, 3.0, 3.3, 4.0])
def test_alloc_counts_match_the_checker(L, d_in, b):
    assert B.cmpq_alloc_counts(d_in, b) == oracle.alloc_counts(d_in, b)


def test_default_counts_and_packed_words_match_the_checker(L):
    import torch

    for d_in, d_out in [(512, 512), (4096, 11008), (28672, 8192), (33, 7)]:
        assert B.cmpq_default_counts(d_in, d_out) == oracle.default_counts(d_in, d_out)
        bits = np.random.default_rng(d_in).integers(2, 5, d_in).astype(np.uint8)
        assert B.cmpq_packed_words(torch.from_numpy(bits), d_out) == oracle.packed_words(bits, d_out)


def test_workspace_sizes(L):
    assert B.cmpq_workspace_bytes(B.OP_COLLECT_STATS, 4096) <= 8 << 20
    for op in range(6):
        assert B.cmpq_workspace_bytes(op, 512, 512) % 256 == 0
        assert B.cmpq_workspace_bytes(op, 0, 512) == 0          # d_in out of range
    assert B.cmpq_workspace_bytes(B.OP_PACK, 512, 1 << 20) == 0   # d_out out of range
    # the fused call needs no more than the outlier step alone: the final fit patches the provisional tables
    assert (B.cmpq_workspace_bytes(B.OP_PROTECT_AND_QUANTIZE, 512, 512)
            == B.cmpq_workspace_bytes(B.OP_EXTRACT_OUTLIERS, 512, 512))
    assert (B.cmpq_workspace_bytes(B.OP_PROTECT_QUANTIZE_PACK, 512, 512)
            > B.cmpq_workspace_bytes(B.OP_PROTECT_AND_QUANTIZE, 512, 512))
    # the whole pass of the largest workload layer (8192 x 28672) fits in 8 bytes per weight of scratch ...
    assert B.cmpq_workspace_bytes(B.OP_PROTECT_QUANTIZE_PACK, 8192, 28672) <= 8 * 8192 * 28672
    # ... while the all-pairs formulation keeps an fp32 error per weight: the answer follows the selected method
    B.cmpq_set_lloyd_assignment(B.ASSIGN_ALL_PAIRS)
    try:
        assert B.cmpq_workspace_bytes(B.OP_EXTRACT_OUTLIERS, 4096, 4096) >= 4 * 4096 * 4096
    finally:
        B.cmpq_set_lloyd_assignment(B.ASSIGN_ORDERED)


def test_bad_arguments_are_refused_on_the_host(L):
    INVALID, UNSUPPORTED, WORKSPACE = 1, 2, 3
    buf = (ctypes.c_char * 4096)()
    p = ctypes.cast(buf, ctypes.c_void_p)
    ws = ctypes.c_void_p((p.value + 255) // 256 * 256)
    # statistic
    assert L.cmpq_collect_stats(p, 0, 4, 8, 8, None, None, ws, 1 << 30, None) == INVALID       # no sumsq
    assert L.cmpq_collect_stats(p, 0, -1, 8, 8, p, None, ws, 1 << 30, None) == INVALID          # n < 0
    assert L.cmpq_collect_stats(p, 0, 4, 8, 7, p, None, ws, 1 << 30, None) == INVALID           # ldx < d_in
    assert L.cmpq_collect_stats(p, 5, 4, 8, 8, p, None, ws, 1 << 30, None) == INVALID           # dtype
    assert L.cmpq_collect_stats(p, 0, 4, 8, 8, p, None, None, 1 << 30, None) == WORKSPACE
    assert L.cmpq_collect_stats(p, 0, 4, 8, 8, p, None, ws, 16, None) == WORKSPACE
    # Algorithm 1 requires b in [2, 4]
    for b in (1.99, 4.01, float("nan")):
        assert L.cmpq_allocate_bits(p, 8, b, 0, p, None, ws, 1 << 30, None) == INVALID
    assert L.cmpq_allocate_bits(p, 8, 3.0, 7, p, None, ws, 1 << 30, None) == INVALID      # mode
    assert L.cmpq_allocate_bits(p, 8, 3.0, 0, p, None, ws, 8, None) == WORKSPACE
    # outliers: counts must be consistent
    args = lambda n_act, n_q, nnz, iters=5, d_out=16: (p, 0, 8, d_out, d_out, p, p, n_act, n_q, iters, p, p, p, nnz, None, ws, 1 << 30, None)
    assert L.cmpq_extract_outliers(*args(9, 0, 9 * 16)) == INVALID
    assert L.cmpq_extract_outliers(*args(1, 7 * 16 + 1, 16 + 7 * 16 + 1)) == INVALID
    assert L.cmpq_extract_outliers(*args(1, 3, 18)) == INVALID                             # nnz mismatch
    assert L.cmpq_extract_outliers(*args(1, 3, 19, iters=-1)) == INVALID
    assert L.cmpq_extract_outliers(*args(1, 3, 19, iters=1001)) == INVALID
    assert L.cmpq_extract_outliers(*args(0, 0, 0, d_out=40000)) == INVALID                 # d_out too large
    # quantizer
    q = lambda sens=None, nnz=0, rows=None, d_out=16, iters=5: (p, 0, 8, d_out, d_out, p, rows, rows, nnz, iters, sens, p, p, None, None, None, ws, 1 << 30, None)
    assert L.cmpq_quantize_layer(*q(sens=ctypes.c_void_p(p.value + 2))) == INVALID           # misaligned sensitivities
    assert L.cmpq_quantize_layer(*q(nnz=3)) == INVALID                                     # list missing
    assert L.cmpq_quantize_layer(*q(d_out=0)) == INVALID
    assert L.cmpq_quantize_layer(*q(iters=2000)) == INVALID
    # eight codes leave in one store: an offset view of a code buffer is refused here, never launched
    qc = lambda codes: (ws, 0, 8, 16, 16, ws, None, None, 0, 5, None, ws, codes, None, None, None, ws, 1 << 30, None)
    assert L.cmpq_quantize_layer(*qc(ctypes.c_void_p(ws.value + 1))) == INVALID
    assert L.cmpq_quantize_layer(*qc(ctypes.c_void_p(ws.value + 4))) == INVALID
    # outlier protection and final fit in one call: the checks of both
    f = lambda n_act=1, n_q=3, nnz=19, lut=p, codes=p, wsb=1 << 30: (p, 0, 8, 16, 16, p, p, n_act, n_q, 5, p, p, p, nnz, lut, codes, None, None, None, ws, wsb, None)
    assert L.cmpq_protect_and_quantize(*f(nnz=18)) == INVALID
    assert L.cmpq_protect_and_quantize(*f(lut=None)) == INVALID
    assert L.cmpq_protect_and_quantize(*f(codes=None)) == INVALID
    assert L.cmpq_protect_and_quantize(*f(wsb=64)) == WORKSPACE
    assert L.cmpq_protect_and_quantize(*f(codes=ctypes.c_void_p(ws.value + 4))) == INVALID   # misaligned codes
    # pack
    assert L.cmpq_pack(p, p, 8, 16, None, p, p, p, ws, 1 << 30, None) == INVALID
    assert L.cmpq_pack(p, p, 8, 16, p, p, p, p, ws, 8, None) == WORKSPACE


def test_assignment_method_is_host_state(L):
    assert L.cmpq_get_lloyd_assignment() == B.ASSIGN_ORDERED          # the default
    assert L.cmpq_set_lloyd_assignment(B.ASSIGN_ALL_PAIRS) == 0
    assert L.cmpq_get_lloyd_assignment() == B.ASSIGN_ALL_PAIRS
    assert L.cmpq_set_lloyd_assignment(7) == 1                        # unknown value: refused, unchanged
    assert L.cmpq_get_lloyd_assignment() == B.ASSIGN_ALL_PAIRS
    assert L.cmpq_set_lloyd_assignment(B.ASSIGN_ORDERED) == 0
    assert B.cmpq_get_lloyd_assignment() == B.ASSIGN_ORDERED


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "_LIB_PATH", "/nonexistent/libcmpq.so")
    with pytest.raises(RuntimeError, match="missing"):
        B.lib()
