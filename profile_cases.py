"""Small, self-ending runs of single C-ABI calls, meant to be captured by a profiler.

    python profile_cases.py lloyd --d-in 1184 --d-out 4096 --bits 3 --launches 3
    python profile_cases.py stats --tokens 32768 --d-in 4096 --launches 3
    python profile_cases.py pack  --d-in 16384 --d-out 8192 --bits 3 --launches 3
    python profile_cases.py outliers --d-in 1184 --d-out 4096 --bits 3 --launches 2
    python profile_cases.py matvec --d-in 8192 --d-out 28672 --budget 2.5 --launches 20
    python profile_cases.py transpose --d-in 16384 --d-out 16384 --launches 10
    python profile_cases.py sweep --config c3_mlp7b --layer 0 --launches 5
    python profile_cases.py stack --config c4_stack7b --budget 3.0
    python profile_cases.py layer --config c3_mlp7b --layer 0 --budget 3.0 --launches 5

`layer` runs the whole pass on one layer of a named workload and prints the time per C-ABI call.
`stack` quantizes every layer of a multi-block workload (all 32 x 7 layers of the Llama-7B-shaped stack) and
prints the total device time of the passes; under torchrun the layers are dealt round-robin to the ranks.

Each case prints the mean CUDA-event time per call; every run holds well under 1 GB on the device.
"""
import argparse
import os
import sys

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2410_13056_b200 import binding as B
from paper_2410_13056_b200 import inputs


def run_layer(a):
    from paper_2410_13056_b200.pipeline import LayerQuantizer

    cfg = inputs.CONFIGS[a.config]
    L = cfg.layers[a.layer]
    seed = inputs.layer_seed(cfg, a.layer)
    W = inputs.make_weight(L.d_in, L.d_out, cfg.dtype, seed, device="cuda")
    X = inputs.make_activations(cfg.n_tokens, L.d_in, cfg.dtype, seed, device="cuda")
    q = LayerQuantizer(L.d_in, L.d_out)
    for _ in range(2):
        q.run(X, W, a.budget, cfg.lloyd_iters)
    torch.cuda.synchronize()
    evs = [dict() for _ in range(a.launches)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(a.launches):
        q.run(X, W, a.budget, cfg.lloyd_iters, events=evs[i], fused=a.fused)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.launches
    params = L.d_in * L.d_out
    print("layer %s[%d] d_in=%d d_out=%d tokens=%d budget=%.2f T=%d: %.3f ms per pass, %.0f Mparams/s"
          % (a.config, a.layer, L.d_in, L.d_out, cfg.n_tokens, a.budget, cfg.lloyd_iters, ms, params / ms / 1e3))
    for name in evs[0]:
        if name == "final_fit_kernels":
            for i, kernel in enumerate(("table", "iterate", "assign")):
                t = sum(e[name][i].elapsed_time(e[name][i + 1]) for e in evs) / a.launches
                print("      final fit, %-12s %.3f ms" % (kernel + " kernel", t))
            continue
        t = sum(e[name][0].elapsed_time(e[name][1]) for e in evs) / a.launches
        print("   %-24s %.3f ms" % (name, t))
    print("   final-fit distance evaluations: %d, inexact rows: %d"
          % (int(q.counters[1].item()), int(q.counters[0].item() & 0xffffffff)))


def run_stack(a):
    """Every layer of a multi-block workload through pipeline.StackQuantizer (weights seeded per layer,
    activations per input width; only the passes are timed); under torchrun the layers are dealt to the ranks."""
    from paper_2410_13056_b200 import sharding
    from paper_2410_13056_b200.pipeline import StackQuantizer

    cfg = inputs.CONFIGS[a.config]
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", torch.cuda.current_device()))
    src = inputs.StackInputs(cfg)
    stack = StackQuantizer(src.shapes(), rank, world)
    seen = set()
    for k in stack.mine:  # one untimed pass per shape: module and buffer set-up
        if stack.shapes[k] not in seen:
            seen.add(stack.shapes[k])
            X, W = src(k)
            stack.quantizer(k).run(X, W, a.budget, cfg.lloyd_iters)
    inexact = [0]

    def on_result(k, r):
        inexact[0] += int(r.inexact_rows.item())

    out = stack.run(src, a.budget, cfg.lloyd_iters, on_result=on_result, timed=True)
    slowest = sharding.max_over_ranks(out["ms"], device="cuda")
    params = out["params"]
    if world > 1:
        t = torch.tensor([float(params)], dtype=torch.float64, device="cuda")
        dist.all_reduce(t)
        params = int(t.item())
        dist.destroy_process_group()
    if rank == 0:
        print("stack %s: %d layers (%d blocks x %d), %.3f G weights, avg %.2f bits, T=%d, %d rank(s): %.1f ms of "
              "passes on the slowest rank, %.0f Mparams/s; inexact rows on rank 0: %d"
              % (a.config, len(src.layers), cfg.repeat, len(cfg.layers), params / 1e9, a.budget, cfg.lloyd_iters,
                 world, slowest, params / slowest / 1e3, inexact[0]))
        for shape, ms in out["ms_by_shape"].items():
            print("   %d x %d: %.3f ms per pass" % (shape[0], shape[1], ms))


def run_sweep(a):
    """All budgets of a workload on one layer: separate passes against run_budgets (statistic computed once)."""
    from paper_2410_13056_b200.pipeline import LayerQuantizer

    cfg = inputs.CONFIGS[a.config]
    L = cfg.layers[a.layer]
    seed = inputs.layer_seed(cfg, a.layer)
    W = inputs.make_weight(L.d_in, L.d_out, cfg.dtype, seed, device="cuda")
    X = inputs.make_activations(cfg.n_tokens, L.d_in, cfg.dtype, seed, device="cuda")
    q = LayerQuantizer(L.d_in, L.d_out)
    budgets = list(cfg.budgets)

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(a.launches):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / a.launches

    separate = timed(lambda: [q.run(X, W, b, cfg.lloyd_iters) for b in budgets])
    stat_only = timed(lambda: q.run_budgets(X, W, budgets, cfg.lloyd_iters, share_fits=False))
    shared = timed(lambda: q.run_budgets(X, W, budgets, cfg.lloyd_iters))
    print("sweep %s[%d] d_in=%d d_out=%d, budgets %s: %.3f ms as separate passes, %.3f ms with the statistic "
          "computed once, %.3f ms with the value tables and provisional fits kept as well"
          % (a.config, a.layer, L.d_in, L.d_out, budgets, separate, stat_only, shared))


def run_matvec(a, dt):
    """The inference product on a random quantized layer (codes are random, so no quantization runs):
    widths split as the rank-form allocation splits them for the budget."""
    from paper_2410_13056_b200.pipeline import QuantizedLinear

    d_in, d_out = a.d_in, a.d_out
    n2, n4 = B.cmpq_alloc_counts(d_in, a.budget)
    n_act, n_q = B.cmpq_default_counts(d_in, d_out)
    g = torch.Generator(device="cuda")
    g.manual_seed(5)
    bits = torch.full((d_in,), 3, dtype=torch.uint8, device="cuda")
    order = torch.randperm(d_in, generator=g, device="cuda")
    bits[order[:n2]] = 2
    bits[order[d_in - n4:]] = 4
    codes = torch.randint(0, 16, (d_in, d_out), dtype=torch.uint8, device="cuda", generator=g)
    codes &= ((1 << bits.int()) - 1).to(torch.uint8)[:, None]
    lut = torch.sort(torch.randn((d_in, 16), device="cuda", generator=g) * 0.02, dim=1).values.contiguous()
    words = B.cmpq_packed_words(bits.cpu(), d_out)
    packed = torch.empty(words, dtype=torch.int32, device="cuda")
    row_off = torch.empty(d_in + 1, dtype=torch.int64, device="cuda")
    perm = torch.empty(d_in, dtype=torch.int32, device="cuda")
    seg = torch.empty(3, dtype=torch.int64, device="cuda")
    B.cmpq_pack(codes, bits, packed, row_off, perm, seg, B.workspace(B.OP_PACK, d_in, d_out))
    nnz = n_act * d_out + n_q
    lin = torch.unique(torch.randint(0, d_in * d_out, (nnz + nnz // 8 + 64,), generator=g, device="cuda"))[:nnz]
    nnz = lin.numel()
    rows, cols = (lin // d_out).int(), (lin % d_out).int()
    vals = (torch.randn(nnz, device="cuda", generator=g) * 0.1).to(inputs.torch_dtype(dt)).view(torch.int16)
    x = torch.randn(d_in, device="cuda", generator=g).to(inputs.torch_dtype(dt))
    layer = QuantizedLinear(packed, row_off, perm, seg, lut, rows, cols, vals, d_out)
    y16 = torch.empty(d_out, dtype=inputs.torch_dtype(dt), device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")  # larger than L2
    for _ in range(3):
        layer.matvec(x, y16)
    torch.cuda.synchronize()
    cold = warm = 0.0
    for _ in range(a.launches):
        flush.zero_()
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record()
        layer.matvec(x, y16)
        e1.record()
        layer.matvec(x, y16)
        e2.record()
        torch.cuda.synchronize()
        cold += e0.elapsed_time(e1) / a.launches
        warm += e1.elapsed_time(e2) / a.launches
    algo = words * 4 + d_in * 64 + nnz * 6 + d_in * 2 + d_out * 4
    print("matvec: d_in=%d d_out=%d avg %.2f bits (%d/%d/%d channels of 2/3/4 bits), nnz=%d; %.1f MB packed, "
          "%.1f MB algorithmic" % (d_in, d_out, a.budget, n2, d_in - n2 - n4, n4, nnz, words * 4 / 1e6, algo / 1e6))
    print("   L2 flushed before the call: %.4f ms (%.0f GB/s); directly repeated: %.4f ms (%.0f GB/s); %d calls"
          % (cold, algo / cold / 1e6, warm, algo / warm / 1e6, a.launches))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["lloyd", "stats", "pack", "outliers", "protect", "layer", "matvec", "stack", "transpose", "sweep"])
    ap.add_argument("--config", default="c2_attn7b")
    ap.add_argument("--layer", type=int, default=0)
    ap.add_argument("--budget", type=float, default=3.0)
    ap.add_argument("--d-in", type=int, default=1184)
    ap.add_argument("--d-out", type=int, default=4096)
    ap.add_argument("--tokens", type=int, default=32768)
    ap.add_argument("--bits", type=int, default=3)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--launches", type=int, default=3)
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f16"])
    ap.add_argument("--fused", action="store_true",
                    help="layer case: outlier protection and final fit through cmpq_protect_and_quantize")
    ap.add_argument("--weighted", action="store_true",
                    help="lloyd case: the sensitivity-weighted fit (random sensitivities)")
    ap.add_argument("--assign", default="ordered", choices=["ordered", "all_pairs"],
                    help="assignment method of the K-means kernels")
    a = ap.parse_args()
    dt = inputs.BF16 if a.dtype == "bf16" else inputs.F16
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    B.cmpq_set_lloyd_assignment(B.ASSIGN_ALL_PAIRS if a.assign == "all_pairs" else B.ASSIGN_ORDERED)
    if a.case == "layer":
        run_layer(a)
        return
    if a.case == "matvec":
        run_matvec(a, dt)
        return
    if a.case == "stack":
        run_stack(a)
        return
    if a.case == "sweep":
        run_sweep(a)
        return
    d_in, d_out = a.d_in, a.d_out
    bits = torch.full((d_in,), a.bits, dtype=torch.uint8, device="cuda")

    if a.case == "transpose":  # a framework's [d_out][d_in] weight into the library's [d_in][d_out]
        src = inputs.make_weight(d_out, d_in, dt, 1, device="cuda")
        dst = torch.empty((d_in, d_out), dtype=src.dtype, device="cuda")
        fn = lambda: B.cmpq_transpose16(src, dst)
        work = "%.1f MB read + %.1f MB written" % (src.numel() * 2 / 1e6, src.numel() * 2 / 1e6)
    elif a.case == "stats":
        X = inputs.make_activations(a.tokens, d_in, dt, 1, device="cuda")
        sumsq = torch.zeros(d_in, dtype=torch.float64, device="cuda")
        ws = B.workspace(B.OP_COLLECT_STATS, d_in)
        fn = lambda: B.cmpq_collect_stats(X, sumsq, ws)
        work = "%.1f MB read" % (X.numel() * 2 / 1e6)
    elif a.case == "pack":
        codes = torch.randint(0, 1 << a.bits, (d_in, d_out), dtype=torch.uint8, device="cuda")
        words = d_in * ((d_out * a.bits + 31) // 32)
        packed = torch.empty(words, dtype=torch.int32, device="cuda")
        row_off = torch.empty(d_in + 1, dtype=torch.int64, device="cuda")
        perm = torch.empty(d_in, dtype=torch.int32, device="cuda")
        seg = torch.empty(3, dtype=torch.int64, device="cuda")
        ws = B.workspace(B.OP_PACK, d_in, d_out)
        fn = lambda: B.cmpq_pack(codes, bits, packed, row_off, perm, seg, ws)
        work = "%.1f MB read + %.1f MB written" % (codes.numel() / 1e6, words * 4 / 1e6)
    else:
        W = inputs.make_weight(d_in, d_out, dt, 1, device="cuda")
        if a.case == "lloyd":
            lut = torch.empty((d_in, 16), dtype=torch.float32, device="cuda")
            codes = torch.empty((d_in, d_out), dtype=torch.uint8, device="cuda")
            counters = torch.zeros(2, dtype=torch.int64, device="cuda")
            ws = B.workspace(B.OP_QUANTIZE_LAYER, d_in, d_out)
            sens = (torch.rand((d_in, d_out), device="cuda") + 0.5) if a.weighted else None
            fn = lambda: B.cmpq_quantize_layer(W, bits, None, None, a.iters, lut, codes, ws, sens=sens,
                                               sweeps=counters[1:2])
            work = "%d channels x %d weights, K=%d, T=%d" % (d_in, d_out, 1 << a.bits, a.iters)
        else:
            n_act, n_q = B.cmpq_default_counts(d_in, d_out)
            nnz = n_act * d_out + n_q
            rows = torch.empty(nnz, dtype=torch.int32, device="cuda")
            cols = torch.empty(nnz, dtype=torch.int32, device="cuda")
            vals = torch.empty(nnz, dtype=torch.int16, device="cuda")
            av = torch.rand(d_in, device="cuda")
            if a.case == "protect":  # outlier protection and final fit in one call
                lut = torch.empty((d_in, 16), dtype=torch.float32, device="cuda")
                codes = torch.empty((d_in, d_out), dtype=torch.uint8, device="cuda")
                ws = B.workspace(B.OP_PROTECT_AND_QUANTIZE, d_in, d_out)
                fn = lambda: B.cmpq_protect_and_quantize(W, av, bits, n_act, n_q, a.iters, rows, cols, vals, lut,
                                                         codes, ws)
            else:
                ws = B.workspace(B.OP_EXTRACT_OUTLIERS, d_in, d_out)
                fn = lambda: B.cmpq_extract_outliers(W, av, bits, n_act, n_q, a.iters, rows, cols, vals, ws)
            work = "%d channels x %d weights, K=%d, T=%d, nnz=%d" % (d_in, d_out, 1 << a.bits, a.iters, nnz)

    fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.launches):
        fn()
    e1.record()
    torch.cuda.synchronize()
    print("%s: %s; %.4f ms per call over %d calls" % (a.case, work, e0.elapsed_time(e1) / a.launches, a.launches))
    if a.case == "lloyd":
        print("distance evaluations per call: %d" % (int(counters[1].item()) // (a.launches + 1)))


if __name__ == "__main__":
    main()
