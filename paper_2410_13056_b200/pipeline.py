"""The whole CMPQ pass for one linear layer as a chain of C-ABI calls.

LayerQuantizer owns the device buffers of one layer shape (outputs and scratch, allocated once
through torch) and enqueues, on the current stream and without host synchronisation, the calls
in the paper's order: statistic (Section 3.2.1) -> Algorithm 1 -> outlier protection
(Section 3.2.2) -> channel-wise K-means and codes -> packing (Section 5.1).  It computes
nothing itself.
"""
from dataclasses import dataclass

import torch

from . import binding as B

# CUDA kernels of this library launched by one LayerQuantizer.run with n_q > 0 and nnz > 0 (the two zero fills
# of the counters and of the statistic's accumulator are torch's and not counted).
# Fused, default assignment (cmpq_protect_quantize_pack): statistic 2 + finalize 1, allocation 1 (two rank cuts
# in one block), outlier step 10 (O_act cut with select start and pack layout, value tables, provisional
# iterations, lower bound, 3 select passes, row counts, row scan, emit), final fit 2 (iterations that patch the
# tables, last assignment that packs) = 16.
# Separate calls: the final fit builds its own tables (row index, tables, iterations, assignment = 4) and the
# packing takes 2 more = 20.  All-pairs assignment: the provisional fit is one kernel and every select pass is
# followed by a digit kernel (outlier step 11), the final fit is row index + one kernel, packing 2 = 19; fused
# the packing still runs as its own step after the fit (layout with the O_act cut, pack 1) = 18.
# With overlap_tables the value tables come from cmpq_sweep_begin on a second stream (table kernel and the
# kernel that empties the cache of fits) and the rest from cmpq_sweep_budget_pack: one kernel more, 17.
def kernels_per_run(assignment=None, fused=False, overlap_tables=False):
    if assignment is None:
        assignment = B.cmpq_get_lloyd_assignment()
    if assignment == B.ASSIGN_ALL_PAIRS:
        return 18 if fused else 19
    if fused and overlap_tables:
        return 17
    return 16 if fused else 20


KERNELS_PER_RUN = 20


@dataclass
class LayerResult:
    """Views of the quantizer's output buffers (overwritten by the next run)."""
    a: torch.Tensor          # [d_in] fp32 activation statistic
    bits: torch.Tensor       # [d_in] uint8 in {2,3,4}
    rows: torch.Tensor       # [nnz] int32 outlier coordinates, sorted by (row, col)
    cols: torch.Tensor       # [nnz] int32
    vals: torch.Tensor       # [nnz] int16 raw 16-bit patterns of the kept weights
    lut: torch.Tensor        # [d_in][16] fp32 centroids
    codes: torch.Tensor      # [d_in][d_out] uint8
    packed: torch.Tensor     # [words] int32 bit streams
    row_off: torch.Tensor    # [d_in+1] int64 word offsets in segment order
    perm: torch.Tensor       # [d_in] int32 channel ids in segment order
    seg_rows: torch.Tensor   # [3] int64 channels per width 2,3,4
    inexact_rows: torch.Tensor  # [1] int32
    sweeps: torch.Tensor     # [1] int64 distance evaluations of the final fit
    d_out: int = 0           # weights per channel (codes may be None)


class LayerQuantizer:
    def __init__(self, d_in, d_out, device="cuda", n_act=None, n_q=None, keep_codes=True):
        """keep_codes=False: the byte codes are never materialised (the last assignment of the final fit
        writes the packed words directly); LayerResult.codes is then None."""
        self.d_in, self.d_out = int(d_in), int(d_out)
        self.keep_codes = bool(keep_codes)
        self.device = torch.device(device)
        da, dq = B.cmpq_default_counts(self.d_in, self.d_out)
        self.n_act = da if n_act is None else int(n_act)
        self.n_q = dq if n_q is None else int(n_q)
        self.nnz = self.n_act * self.d_out + self.n_q
        dev = self.device
        self.ws = None
        self._ensure_ws()
        self.sumsq = torch.empty(self.d_in, dtype=torch.float64, device=dev)
        self.a = torch.empty(self.d_in, dtype=torch.float32, device=dev)
        self.bits = torch.empty(self.d_in, dtype=torch.uint8, device=dev)
        self.rows = torch.empty(self.nnz, dtype=torch.int32, device=dev)
        self.cols = torch.empty(self.nnz, dtype=torch.int32, device=dev)
        self.vals = torch.empty(self.nnz, dtype=torch.int16, device=dev)
        self.lut = torch.empty((self.d_in, B.LUT_STRIDE), dtype=torch.float32, device=dev)
        self.codes = torch.empty((self.d_in, self.d_out), dtype=torch.uint8, device=dev) if keep_codes else None
        max_words = self.d_in * ((self.d_out * 4 + 31) // 32)
        self.packed = torch.empty(max_words, dtype=torch.int32, device=dev)
        self.row_off = torch.empty(self.d_in + 1, dtype=torch.int64, device=dev)
        self.perm = torch.empty(self.d_in, dtype=torch.int32, device=dev)
        self.seg_rows = torch.empty(3, dtype=torch.int64, device=dev)
        self.counters = torch.zeros(4, dtype=torch.int64, device=dev)

    def _ensure_ws(self):
        """One scratch buffer large enough for every call of the pass.  The size depends on the assignment
        method selected in the library (the all-pairs method keeps an fp32 error per weight), so it is
        checked again before every run."""
        need = max(B.cmpq_workspace_bytes(op, self.d_in, self.d_out)
                   for op in list(range(6)) + [B.OP_PROTECT_QUANTIZE_PACK])
        if self.ws is None or self.ws.numel() < need:
            self.ws = torch.empty(max(need, 256), dtype=torch.uint8, device=self.device)
            self._graphs = {}  # captured graphs hold the old buffer's address

    def check_finite(self):
        """Waits for the last run and raises binding.CmpqError (status 6) if its activations or weights
        held a NaN or an infinity (the run's outputs are then unspecified)."""
        B.cmpq_check_finite(self.nonfinite)

    def packed_words(self, avg_bits):
        """Words the rank-form allocation produces for this budget (no device read needed)."""
        n2, n4 = B.cmpq_alloc_counts(self.d_in, avg_bits)
        n3 = self.d_in - n2 - n4
        w = lambda c: (self.d_out * c + 31) // 32
        return n2 * w(2) + n3 * w(3) + n4 * w(4)

    def run_budgets(self, X, W, budgets, lloyd_iters, on_result=None, share_fits=True):
        """The pass for several average budgets on the same layer (the paper's budget sweeps: any new
        constraint means quantizing again).  Three things do not depend on the budget and are computed once:
        the activation statistic, the value tables of the channels (cmpq_sweep_begin) and the provisional
        fit of a channel at a given width, which is kept the first time a budget needs it
        (cmpq_sweep_budget).  Every budget re-runs Algorithm 1, the remaining provisional fits, the
        selection, the final fit and the packing; each budget's outputs are exactly those of a separate
        run().  share_fits=False shares the statistic only.  The output buffers are reused, so
        on_result(budget, result) is called after each budget's work has been enqueued (copy what you need
        there, on the same stream).  Returns the last result."""
        result = None
        cache = None
        if share_fits and B.cmpq_get_lloyd_assignment() == B.ASSIGN_ORDERED:
            if getattr(self, "_sweep_cache", None) is None:
                self._sweep_cache = torch.empty(B.cmpq_sweep_cache_bytes(self.d_in, self.d_out), dtype=torch.uint8,
                                                device=self.device)
            cache = self._sweep_cache
            B.cmpq_sweep_begin(W, lloyd_iters, cache)
        for k, b in enumerate(budgets):
            result = self.run(X, W, b, lloyd_iters, reuse_statistic=k > 0, sweep_cache=cache)
            if on_result is not None:
                on_result(b, result)
        return result

    def run(self, X, W, avg_bits, lloyd_iters, events=None, fused=None, reuse_statistic=False, sweep_cache=None,
            overlap_tables=False):
        """Enqueue the pass for calibration activations X [n][d_in] and weights W [d_in][d_out].
        reuse_statistic: keep the statistic `a` of the previous run on the same X (see run_budgets).
        sweep_cache: a cache prepared by cmpq_sweep_begin for W (see run_budgets).
        fused (default: True unless events are asked for): outlier protection, final fit and packing through
        cmpq_protect_quantize_pack, which derives the final fit's value tables from the provisional fit's
        and lets the last assignment write the packed words; otherwise cmpq_extract_outliers,
        cmpq_quantize_layer and cmpq_pack one after the other (same results; needs keep_codes).
        overlap_tables (fused runs of the default assignment without events): the value tables depend on the
        weights alone, so they are built on a second stream (cmpq_sweep_begin into a cache this object keeps)
        while the current stream computes the statistic and the allocation; the streams join before
        cmpq_sweep_budget_pack.  Same results; one table set more of device memory.  events (optional dict) receives a (start, end) CUDA event pair per C-ABI call and,
        when not fused, under "final_fit_kernels" the four events around the three kernels of the
        final K-means."""
        if fused is None:
            fused = events is None or not self.keep_codes
        assert fused or self.keep_codes
        assert W.shape == (self.d_in, self.d_out) and X.shape[1] == self.d_in

        def call(name, fn, *args, **kw):
            if events is None:
                fn(*args, **kw)
                return
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn(*args, **kw)
            e1.record()
            events[name] = (e0, e1)

        self._ensure_ws()
        self.counters.zero_()
        inexact = self.counters[0:1].view(torch.int32)[0:1]
        sweeps = self.counters[1:2]
        nonfinite = self.nonfinite = self.counters[2:3].view(torch.int32)[0:1]
        side = None
        if (overlap_tables and fused and events is None and sweep_cache is None and not reuse_statistic
                and B.cmpq_get_lloyd_assignment() == B.ASSIGN_ORDERED):
            if getattr(self, "_overlap_cache", None) is None:
                self._overlap_cache = torch.empty(B.cmpq_sweep_cache_bytes(self.d_in, self.d_out), dtype=torch.uint8,
                                                  device=self.device)
                self._side_stream = torch.cuda.Stream(device=self.device)
            sweep_cache, side = self._overlap_cache, self._side_stream
        if not reuse_statistic:
            self.sumsq.zero_()
            if side is not None:
                # The previous pass may still be reading the cache.  The fork comes directly before the
                # statistic: both kernels then depend on the same predecessor and the statistic, enqueued
                # first, gets its blocks placed first (the other order leaves nothing to overlap).
                side.wait_stream(torch.cuda.current_stream())
            call("cmpq_collect_stats", B.cmpq_collect_stats, X, self.sumsq, self.ws, nonfinite=nonfinite)
            if side is not None:  # enqueued after the statistic so that its blocks are placed first
                with torch.cuda.stream(side):
                    B.cmpq_sweep_begin(W, lloyd_iters, sweep_cache, nonfinite=nonfinite)
            call("cmpq_finalize_stats", B.cmpq_finalize_stats, self.sumsq, self.a)
        call("cmpq_allocate_bits", B.cmpq_allocate_bits, self.a, avg_bits, B.ALLOC_RANK, self.bits, None,
             self.ws)
        if side is not None:
            torch.cuda.current_stream().wait_stream(side)
        if sweep_cache is not None and fused:
            call("cmpq_sweep_budget_pack", B.cmpq_sweep_budget_pack, W, self.a, self.bits, self.n_act, self.n_q,
                 lloyd_iters, self.rows, self.cols, self.vals, self.lut, self.codes, self.packed, self.row_off,
                 self.perm, self.seg_rows, sweep_cache, self.ws, inexact_rows=inexact, sweeps=sweeps)
        elif sweep_cache is not None:
            call("cmpq_sweep_budget", B.cmpq_sweep_budget, W, self.a, self.bits, self.n_act, self.n_q, lloyd_iters,
                 self.rows, self.cols, self.vals, self.lut, self.codes, sweep_cache, self.ws,
                 inexact_rows=inexact, sweeps=sweeps)
            call("cmpq_pack", B.cmpq_pack, self.codes, self.bits, self.packed, self.row_off, self.perm,
                 self.seg_rows, self.ws)
        elif fused:  # outlier protection, final fit and packing in one call
            call("cmpq_protect_quantize_pack", B.cmpq_protect_quantize_pack, W, self.a, self.bits, self.n_act,
                 self.n_q, lloyd_iters, self.rows, self.cols, self.vals, self.lut, self.codes, self.packed,
                 self.row_off, self.perm, self.seg_rows, self.ws, inexact_rows=inexact, sweeps=sweeps,
                 nonfinite=nonfinite)
        else:
            self._protect_then_quantize(call, W, lloyd_iters, events, inexact, sweeps)
            call("cmpq_pack", B.cmpq_pack, self.codes, self.bits, self.packed, self.row_off, self.perm,
                 self.seg_rows, self.ws)
        words = self.packed_words(avg_bits)
        return LayerResult(self.a, self.bits, self.rows, self.cols, self.vals, self.lut, self.codes,
                           self.packed[:words], self.row_off, self.perm, self.seg_rows, inexact, sweeps, self.d_out)

    def _protect_then_quantize(self, call, W, lloyd_iters, events, inexact, sweeps):
        call("cmpq_extract_outliers", B.cmpq_extract_outliers, W, self.a, self.bits, self.n_act, self.n_q,
             lloyd_iters, self.rows, self.cols, self.vals, self.ws)
        if events is not None and B.cmpq_get_lloyd_assignment() == B.ASSIGN_ORDERED:
            # the three kernels of the final fit, timed separately
            phase = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            B.cmpq_lloyd_phase_events(phase)
            events["final_fit_kernels"] = phase
        call("cmpq_quantize_layer", B.cmpq_quantize_layer, W, self.bits, self.rows, self.cols, lloyd_iters,
             self.lut, self.codes, self.ws, inexact_rows=inexact, sweeps=sweeps)

    def run_graphed(self, X, W, avg_bits, lloyd_iters, overlap_tables=False):
        """The same pass replayed from a CUDA graph: the launches of a pass are short enough for launch
        overhead to show, and nothing in the pass depends on values read back by the host.  The graph is
        captured on the first call for a given (X, W, budget, iterations) and replayed afterwards; X
        and W must keep their addresses (their contents may change).  Results as in run()."""
        key = (X.data_ptr(), W.data_ptr(), tuple(X.shape), float(avg_bits), int(lloyd_iters),
               B.cmpq_get_lloyd_assignment(), bool(overlap_tables))
        if not hasattr(self, "_graphs"):
            self._graphs = {}
        entry = self._graphs.get(key)
        if entry is None:
            cur = torch.cuda.current_stream()
            side = torch.cuda.Stream()
            side.wait_stream(cur)
            with torch.cuda.stream(side):  # first-use initialisation must not be captured
                self.run(X, W, avg_bits, lloyd_iters, overlap_tables=overlap_tables)
            cur.wait_stream(side)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                result = self.run(X, W, avg_bits, lloyd_iters, overlap_tables=overlap_tables)
            entry = (graph, result)
            self._graphs[key] = entry
        entry[0].replay()
        return entry[1]

    # ---- host-buffer entry: the same pass with the copies a caller holding host tensors pays ----
    def make_host_outputs(self, avg_bits):
        """Pinned host tensors for everything a caller stores for one quantized layer."""
        words = self.packed_words(avg_bits)
        pin = lambda t, n=None: torch.empty(t.shape if n is None else (n,), dtype=t.dtype, pin_memory=True)
        return {"bits": pin(self.bits), "rows": pin(self.rows), "cols": pin(self.cols), "vals": pin(self.vals),
                "lut": pin(self.lut), "packed": pin(self.packed, words), "row_off": pin(self.row_off),
                "perm": pin(self.perm), "seg_rows": pin(self.seg_rows), "counters": pin(self.counters)}

    def run_host(self, X_host, W_host, avg_bits, lloyd_iters, host_out):
        """X_host, W_host: pinned host tensors.  Copies them in, runs the pass, copies the stored
        representation (not the byte codes) back into host_out and waits for it."""
        if not hasattr(self, "_Xd") or self._Xd.shape != X_host.shape or self._Xd.dtype != X_host.dtype:
            self._Xd = torch.empty(X_host.shape, dtype=X_host.dtype, device=self.device)
            self._Wd = torch.empty(W_host.shape, dtype=W_host.dtype, device=self.device)
        self._Xd.copy_(X_host, non_blocking=True)
        self._Wd.copy_(W_host, non_blocking=True)
        r = self.run_graphed(self._Xd, self._Wd, avg_bits, lloyd_iters)
        src = {"bits": r.bits, "rows": r.rows, "cols": r.cols, "vals": r.vals, "lut": r.lut, "packed": r.packed,
               "row_off": r.row_off, "perm": r.perm, "seg_rows": r.seg_rows, "counters": self.counters}
        for k, t in host_out.items():
            t.copy_(src[k], non_blocking=True)
        torch.cuda.current_stream().synchronize()
        return host_out


class StackQuantizer:
    """The pass over a list of independent linear layers (Section 3.2.1 of the paper quantizes layer by
    layer, so a transformer stack is just many such layers): this rank's share of them, one after the
    other on the current stream, with one LayerQuantizer (output buffers and scratch) per distinct shape.

    shapes: (d_in, d_out) of every layer of the stack, in order.  With world > 1 the layers are dealt
    round-robin to the ranks (sharding.layers_of_rank); nothing is exchanged between ranks.
    quantizer_factory(d_in, d_out) builds the per-shape quantizer (default: LayerQuantizer on `device`)."""

    def __init__(self, shapes, rank=0, world=1, device="cuda", quantizer_factory=None):
        from . import sharding

        self.shapes = [(int(d_in), int(d_out)) for d_in, d_out in shapes]
        self.rank, self.world = int(rank), int(world)
        self.mine = sharding.layers_of_rank(len(self.shapes), self.rank, self.world)
        self._factory = quantizer_factory or (lambda d_in, d_out: LayerQuantizer(d_in, d_out, device=device))
        self._quantizers = {}

    def quantizer(self, k):
        """The quantizer that serves layer k (shared by all layers of that shape)."""
        shape = self.shapes[k]
        if shape not in self._quantizers:
            self._quantizers[shape] = self._factory(*shape)
        return self._quantizers[shape]

    def params(self):
        """Weights in this rank's layers."""
        return sum(self.shapes[k][0] * self.shapes[k][1] for k in self.mine)

    def run(self, inputs_of, avg_bits, lloyd_iters, on_result=None, timed=False, graphed=False, overlap_tables=False):
        """inputs_of(k) -> (X [n][d_in], W [d_in][d_out]) for layer k of this rank (called right before
        the layer's pass; preparing the inputs is the caller's work and is not timed).  on_result(k, result)
        is called after layer k's pass has been enqueued; the result's buffers are reused by the next layer
        of the same shape, so copy what is kept there (on the same stream).  timed: CUDA events around every
        pass; the returned dict then holds "ms" (the sum over this rank's passes) and "ms_by_shape".
        graphed: passes through LayerQuantizer.run_graphed (inputs_of must then return tensors at fixed
        addresses per shape).  overlap_tables: as in LayerQuantizer.run.  Returns {"layers", "params"[, "ms", "ms_by_shape"]}."""
        pairs = []
        for k in self.mine:
            X, W = inputs_of(k)
            q = self.quantizer(k)
            if timed:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
            extra = {"overlap_tables": True} if overlap_tables else {}  # (a stand-in quantizer need not know the option)
            r = (q.run_graphed if graphed else q.run)(X, W, avg_bits, lloyd_iters, **extra)
            if timed:
                e1.record()
                pairs.append((k, e0, e1))
            if on_result is not None:
                on_result(k, r)
        out = {"layers": len(self.mine), "params": self.params()}
        if timed:
            torch.cuda.current_stream().synchronize()
            by_shape = {}
            for k, e0, e1 in pairs:
                by_shape.setdefault(self.shapes[k], []).append(e0.elapsed_time(e1))
            out["ms"] = sum(sum(v) for v in by_shape.values())
            out["ms_by_shape"] = {shape: sum(v) / len(v) for shape, v in by_shape.items()}
        return out


class QuantizedLinear:
    """A quantized layer held the way inference reads it (Section 6 of the paper): packed 2/3/4-bit
    segments, look-up tables and the outliers grouped by column.  matvec(x) enqueues y = x (W_q + O)
    for one token; it computes nothing itself."""

    def __init__(self, packed, row_off, perm, seg_rows, lut, rows, cols, vals, d_out):
        self.d_in, self.d_out = int(lut.shape[0]), int(d_out)
        self.packed, self.row_off, self.perm, self.seg_rows, self.lut = packed, row_off, perm, seg_rows, lut
        dev = lut.device
        nnz = 0 if rows is None else rows.numel()
        self.col_ptr = self.c_rows = self.c_vals = None
        if nnz:
            self.col_ptr = torch.empty(self.d_out + 1, dtype=torch.int64, device=dev)
            self.c_rows = torch.empty(nnz, dtype=torch.int32, device=dev)
            self.c_vals = torch.empty(nnz, dtype=torch.int16, device=dev)
            B.cmpq_outliers_by_column(rows, cols, vals, self.d_out, self.col_ptr, self.c_rows, self.c_vals,
                                      B.workspace(B.OP_OUTLIERS_BY_COLUMN, 1, self.d_out, device=dev))
        self.ws = B.workspace(B.OP_MATVEC, self.d_in, self.d_out, device=dev)
        self.y = torch.empty(self.d_out, dtype=torch.float32, device=dev)

    @classmethod
    def from_result(cls, r: "LayerResult"):
        return cls(r.packed, r.row_off, r.perm, r.seg_rows, r.lut, r.rows, r.cols, r.vals, r.d_out)

    def packed_bytes(self):
        return self.packed.numel() * 4

    def matvec(self, x, y16=None):
        """x: [d_in] fp16/bf16 on the device.  Returns the fp32 result buffer (overwritten by the next call)."""
        B.cmpq_matvec(self.packed, self.row_off, self.perm, self.seg_rows, self.lut, x, self.col_ptr, self.c_rows,
                      self.c_vals, self.y, y16, self.ws)
        return self.y
