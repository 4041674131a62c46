"""Timing of the supernet-side forms (Sec. 3.1 of the ELSA paper: shared weight, dynamic masking).

    python bench_supernet.py [--out bench_out/supernet.json]

(a) elsa_nm_compress_levels: all levels {1,2,4,8}:8 of a weight from one read, against one
    elsa_nm_compress call per level (GB/s counts the dense weight once plus every packed form
    written).
(b) elsa_nm_linear_masked (dense shared weight + level, no packed copy) against elsa_nm_compress +
    elsa_nm_linear on the DeiT-B layer shapes at batch 256, bf16.
CUDA-event medians of 7 repetitions, 512 MB written between repetitions to flush L2.
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


def timed(fn, flush, reps=7):
    out = []
    for _ in range(reps):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        out.append(e0.elapsed_time(e1))
    return statistics.median(out)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default="bench_out/supernet.json")
    args = ap.parse_args()
    dtype = torch.bfloat16
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    levels = [1, 2, 4, 8]
    results = []
    for out, in_ in [(768, 768), (2304, 768), (3072, 768), (768, 3072)]:
        W = synth.randn((out, in_), 11 + out, synth.W_STD, dtype, "cuda")
        lib.elsa_nm_compress_levels(W, levels, 8)
        packed = [lib.alloc_packed(out, in_, N, 8, dtype) for N in levels]
        ms_all = timed(lambda: lib.elsa_nm_compress_levels(W, levels, 8), flush)
        ms_each = timed(lambda: [lib.elsa_nm_compress(W, N, 8, vals=v, idx=i) for N, (v, i) in zip(levels, packed)], flush)
        nbytes = W.numel() * 2 + sum(v.numel() * 2 + (i.numel() * 4 if i is not None else 0) for v, i in packed)
        rec = {"op": "compress_levels", "out": out, "in": in_, "levels": levels, "ms_one_pass": ms_all,
               "ms_per_level_calls": ms_each, "gbs_one_pass": nbytes / ms_all / 1e6}
        results.append(rec)
    rows = 256 * 197
    for name, in_, out in [("qkv", 768, 2304), ("proj", 768, 768), ("fc1", 768, 3072), ("fc2", 3072, 768)]:
        X = synth.randn((rows, in_), 21, synth.X_STD, dtype, "cuda")
        W = synth.randn((out, in_), 22, synth.W_STD, dtype, "cuda")
        b = synth.randn((out,), 23, synth.B_STD, dtype, "cuda")
        Y = torch.empty((rows, out), dtype=dtype, device="cuda")
        for N in levels:
            ws = lib.alloc_workspace(lib.elsa_workspace_bytes(rows, in_, out, N, 8, lib.BF16))
            vals, idx = lib.alloc_packed(out, in_, N, 8, dtype)

            def packed_path():
                lib.elsa_nm_compress(W, N, 8, vals=vals, idx=idx)
                lib.elsa_nm_linear(X, vals, idx, b, out, in_, N, 8, Y=Y, workspace=ws)

            def masked_path():
                lib.elsa_nm_linear_masked(X, W, b, N, 8, Y=Y, workspace=ws)

            packed_path(); masked_path()
            results.append({"op": "linear_masked", "layer": name, "rows": rows, "in": in_, "out": out, "level": "%d:8" % N,
                            "ms_masked": timed(masked_path, flush), "ms_compress_then_linear": timed(packed_path, flush)})
        del X, Y
    os.makedirs(os.path.dirname(args.out) or ".", exist_ok=True)
    json.dump(results, open(args.out, "w"), indent=1)
    for r in results:
        print(json.dumps(r))


if __name__ == "__main__":
    main()
