"""Shape / sparsity sweep of elsa_nm_linear and elsa_nm_compress on one GPU.

    python bench_sweep.py [--out bench_out/sweep.json] [--reps 5] [--quick]

rows in {4096, 16384, 65536} x (K, O) in {(768,768), (768,3072), (3072,768), (1024,4096), (4096,1024)}
x level in {1:4, 2:4, 1:8, 2:8, 4:8, 1:16, 2:16, 4:16, 8:16} x {fp16, bf16}: per point the median
CUDA-event time of elsa_nm_linear (weight-image rebuild + GEMM) with L2 flushed between repetitions
(small points are otherwise L2-resident), dense-equivalent and kept TFLOP/s, algorithmic GB/s and
the fraction of the layer's roofline; per weight shape, level and dtype the time and GB/s (bytes
read + written) of elsa_nm_compress.  For scale, under the same timing: an empty kernel (what the method itself
costs) and the library's dense product of every (rows, K, O) in bf16 (torch.matmul, i.e. cuBLAS; context, not a
path of this library).  Writes a JSON list and prints a short table.
"""
from __future__ import annotations

import argparse
import json
import statistics

import torch

import os
import sys

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2409_09708_b200 import binding as lib
from paper_2409_09708_b200 import synth


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), "measured"
    return 6650.0, 1590.0, "fallback"


def timed(fn, reps, flush):
    out = []
    for _ in range(reps):
        flush.fill_(1)                       # 512 MB written: evicts the 126 MB L2
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        out.append(e0.elapsed_time(e1))
    return statistics.median(out), min(out)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default="bench_out/sweep.json")
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--quick", action="store_true", help="rows = 4096 only")
    ap.add_argument("--summary", default=None, help="also write a short markdown summary to this path")
    args = ap.parse_args()
    hbm, tf, kind = load_peaks()
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    results = []
    for dt in ("f16", "bf16"):
        dtype = synth.torch_dtype(dt)
        code = lib.dtype_code(dtype)
        cache = {}
        for l in synth.sweep():
            if args.quick and l.rows != synth.SWEEP_ROWS[0]:
                continue
            wkey = (l.in_, l.out, l.N, l.M)
            if wkey not in cache:
                W = synth.randn((l.out, l.in_), l.seed_w, synth.W_STD, dtype, "cuda")
                vals, idx = lib.alloc_packed(l.out, l.in_, l.N, l.M, dtype)
                lib.elsa_nm_compress(W, l.N, l.M, vals=vals, idx=idx)
                ms, best = timed(lambda: lib.elsa_nm_compress(W, l.N, l.M, vals=vals, idx=idx), args.reps, flush)
                nbytes = W.numel() * 2 + vals.numel() * 2 + (idx.numel() * 4 if idx is not None else 0)
                results.append({"op": "compress", "dtype": dt, "in": l.in_, "out": l.out, "level": "%d:%d" % (l.N, l.M),
                                "ms": ms, "ms_min": best, "bytes": nbytes, "gbs": nbytes / ms / 1e6})
                cache[wkey] = (vals, idx)
            vals, idx = cache[wkey]
            X = synth.randn((l.rows, l.in_), l.seed_x, synth.X_STD, dtype, "cuda")
            b = synth.randn((l.out,), l.seed_b, synth.B_STD, dtype, "cuda")
            Y = torch.empty((l.rows, l.out), dtype=dtype, device="cuda")
            ws = lib.alloc_workspace(lib.elsa_workspace_bytes(l.rows, l.in_, l.out, l.N, l.M, code))
            run = lambda: lib.elsa_nm_linear(X, vals, idx, b, l.out, l.in_, l.N, l.M, Y=Y, workspace=ws, dev_status=status)
            run(); run()
            ms, best = timed(run, args.reps, flush)
            alg = X.numel() * 2 + Y.numel() * 2 + vals.numel() * 2 + (idx.numel() * 4 if idx is not None else 0) + l.out * 2
            roof = max(l.kept_flops / (tf * 1e12), alg / (hbm * 1e9)) * 1e3
            results.append({"op": "linear", "dtype": dt, "rows": l.rows, "in": l.in_, "out": l.out,
                            "level": "%d:%d" % (l.N, l.M), "ms": ms, "ms_min": best,
                            "dense_equiv_tflops": l.dense_equiv_flops / ms / 1e9, "kept_tflops": l.kept_flops / ms / 1e9,
                            "algorithmic_gbs": alg / ms / 1e6, "roofline_ms": roof, "roofline_frac": roof / ms,
                            "bound": "tensor" if l.kept_flops / (tf * 1e12) >= alg / (hbm * 1e9) else "hbm"})
            del X, Y
    # scale: what the timing method costs for an empty kernel, and the library's dense GEMM on the same shapes
    tiny = torch.zeros(32, device="cuda")
    tiny.add_(1)
    ms, best = timed(lambda: tiny.add_(1), max(args.reps, 9), flush)
    results.append({"op": "empty_kernel", "ms": ms, "ms_min": best})
    for rows in ([synth.SWEEP_ROWS[0]] if args.quick else synth.SWEEP_ROWS):
        for K, O in synth.SWEEP_SHAPES:
            X = synth.randn((rows, K), 1, synth.X_STD, torch.bfloat16, "cuda")
            W = synth.randn((O, K), 2, synth.W_STD, torch.bfloat16, "cuda")
            Y = torch.empty((rows, O), dtype=torch.bfloat16, device="cuda")
            run = lambda: torch.matmul(X, W.t(), out=Y)
            run(); run()
            ms, best = timed(run, args.reps, flush)
            results.append({"op": "library_dense", "dtype": "bf16", "rows": rows, "in": K, "out": O, "ms": ms, "ms_min": best})
            del X, Y
    assert int(status.item()) == 0
    os.makedirs(os.path.dirname(args.out) or ".", exist_ok=True)
    json.dump({"peaks": {"hbm_gbs": hbm, "bf16_tflops": tf, "kind": kind}, "results": results}, open(args.out, "w"), indent=0)
    lin = [r for r in results if r["op"] == "linear"]
    cmp_ = [r for r in results if r["op"] == "compress"]
    print("linear points: %d, median roofline fraction %.3f, min %.3f, max %.3f" % (
        len(lin), statistics.median(r["roofline_frac"] for r in lin), min(r["roofline_frac"] for r in lin),
        max(r["roofline_frac"] for r in lin)))
    print("compress points: %d, median GB/s %.0f, max %.0f" % (
        len(cmp_), statistics.median(r["gbs"] for r in cmp_), max(r["gbs"] for r in cmp_)))


    if args.summary:
        write_summary(args.summary, hbm, tf, kind, lin, cmp_, results)


def write_summary(path, hbm, tf, kind, lin, cmp_, results):
    med = statistics.median
    out = ["# Shape / sparsity sweep (%d linear points, %d compress points) -- summary" % (len(lin), len(cmp_)), "",
           "Command: `python bench_sweep.py --out bench_out/sweep.json --summary <this file>` (B200;",
           "median of 5 CUDA-event timings per point, 512 MB written between repetitions to flush the 126 MB L2;",
           "time = weight-image rebuild + GEMM of `elsa_nm_linear` under the automatic dispatch).",
           "Peaks (%s): %.1f GB/s, %.1f TFLOP/s." % (kind, hbm, tf), "",
           "Median fraction of the per-point roofline, max(kept FLOPs / tensor peak, algorithmic bytes / HBM peak),",
           "by level and rows, both dtypes and all five (K, O) shapes:", "",
           "| level | rows 4096 | rows 16384 | rows 65536 |", "|---|---|---|---|"]
    for lv in ["%d:%d" % nm for nm in synth.SWEEP_LEVELS]:
        row = [lv]
        for R in synth.SWEEP_ROWS:
            v = [r["roofline_frac"] for r in lin if r["level"] == lv and r["rows"] == R]
            row.append("%.2f" % med(v) if v else "-")
        out.append("| " + " | ".join(row) + " |")
    out += ["", "Dense-equivalent TFLOP/s at rows 65536, median over dtypes, per (K, O) for 2:8 / 4:8:", ""]
    for K, O in synth.SWEEP_SHAPES:
        vals = []
        for lv in ("2:8", "4:8"):
            v = [r["dense_equiv_tflops"] for r in lin if r["rows"] == 65536 and r["in"] == K and r["out"] == O and r["level"] == lv]
            vals.append("%.0f" % med(v) if v else "-")
        out.append("- K=%d, O=%d: %s / %s" % (K, O, vals[0], vals[1]))
    out += ["", "elsa_nm_compress (bytes read + written / time, cold L2): median %.0f GB/s, best %.0f GB/s; the weights"
            % (med(r["gbs"] for r in cmp_), max(r["gbs"] for r in cmp_)),
            "are 1.2-8.4 MB, so a single launch lasts a few microseconds and is latency-bound; tables of weights go",
            "through `elsa_vit_compress`, one launch for all of them.", ""]
    empty = [r for r in results if r["op"] == "empty_kernel"]
    dense = [r for r in results if r["op"] == "library_dense"]
    if empty and dense:
        out += ["For scale, same timing method: an empty kernel reads %.1f us (the floor every point carries).  Microseconds,"
                % (empty[0]["ms"] * 1e3),
                "bf16: the library's dense product (torch.matmul) / this library at 2:8 / at 4:8, per shape and rows:", "",
                "| K, O | " + " | ".join("rows %d" % R for R in synth.SWEEP_ROWS) + " |", "|---|" + "---|" * len(synth.SWEEP_ROWS)]
        for K, O in synth.SWEEP_SHAPES:
            row = ["%d, %d" % (K, O)]
            for R in synth.SWEEP_ROWS:
                d = [r["ms"] * 1e3 for r in dense if r["rows"] == R and r["in"] == K and r["out"] == O]
                ours = []
                for lv in ("2:8", "4:8"):
                    v = [r["ms"] * 1e3 for r in lin if r["rows"] == R and r["in"] == K and r["out"] == O
                         and r["level"] == lv and r["dtype"] == "bf16"]
                    ours.append("%.1f" % v[0] if v else "-")
                row.append("%s / %s / %s" % ("%.1f" % d[0] if d else "-", ours[0], ours[1]))
            out.append("| " + " | ".join(row) + " |")
        out.append("")
    with open(path, "w") as f:
        f.write("\n".join(out))


if __name__ == "__main__":
    main()
