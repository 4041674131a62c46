"""Runs one N:M linear layer a few times through the C ABI: a small, bounded case for profilers.

    python bench_case.py --rows 50432 --in 768 --out 3072 --level 2:8 \
        --dtype bf16 --reps 3

Prints one JSON line with the CUDA-event time of each repetition (compress once, then `reps`
calls of elsa_nm_linear), the layer's algorithmic bytes and kept FLOPs.

    python bench_case.py --compress-table deit_b_stack_b256 --reps 3

runs elsa_vit_compress over the weights of a workload table instead (weights only, no activations).

    python bench_case.py --backward --rows 50432 --in 768 --out 3072 --level 2:8 --reps 5

times elsa_nm_linear_backward on that layer: dX alone, dW alone, db alone and all three in one call.

    python bench_case.py --attention --images 256 --tokens 197 --heads 12 --reps 5

times elsa_attention alone (qkv of that many images in, a out).
"""
from __future__ import annotations

import argparse
import json

import torch

import os
import sys

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2409_09708_b200 import binding as lib
from paper_2409_09708_b200 import synth


def compress_table(workload, reps):
    layers, dt = synth.workload(workload)
    dtype = synth.torch_dtype(dt)
    dev = []
    for l in layers:
        W = synth.randn((l.out, l.in_), l.seed_w, synth.W_STD, dtype, device="cuda")
        vals, idx = lib.alloc_packed(l.out, l.in_, l.N, l.M, dtype)
        dev.append(dict(W=W, vals=vals, idx=idx, N=l.N, M=l.M))
    table = lib.make_weight_table(dev)
    code = lib.dtype_code(dtype)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    times = []
    for rep in range(reps):
        flush.fill_(rep)                          # the weights leave L2 between repetitions
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        lib.elsa_vit_compress(table, code)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    nbytes = sum(l.out * l.in_ * 2 + lib.elsa_nm_values_bytes(l.out, l.in_, l.N, l.M, code) +
                 lib.elsa_nm_index_bytes(l.out, l.in_, l.N, l.M) for l in layers)
    print(json.dumps({"workload": workload, "weights": len(layers), "ms": times, "bytes_read_and_written": nbytes}))


def int8_case(args):
    """One layer in the INT8 form: seeded int8 activations and weights, per-feature scales, 16-bit output."""
    N, M = (int(v) for v in args.level.split(":"))
    dtype = synth.torch_dtype(args.dtype)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    X = torch.randint(-128, 128, (args.rows, args.in_), dtype=torch.int8, device="cuda", generator=gen)
    W = torch.randint(-128, 128, (args.out, args.in_), dtype=torch.int8, device="cuda", generator=gen)
    w_scale = torch.rand(args.out, device="cuda", generator=gen) * 1e-3 + 1e-4
    bias = synth.randn((args.out,), 3, synth.B_STD, dtype, device="cuda")
    vals, idx = lib.elsa_nm_compress_i8(W, N, M)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    times = []
    for rep in range(args.reps):
        flush.fill_(rep)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        lib.elsa_nm_linear_i8(X, 0.02, vals, idx, w_scale, bias, args.out, args.in_, N, M, dtype, dev_status=status)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    assert int(status.item()) == 0
    bits = {4: 2, 8: 3, 16: 4}[M]
    idx_bytes = 0 if N == M else args.out * (-(-(args.in_ // M * N * bits) // 32)) * 4
    alg = args.rows * args.in_ + args.rows * args.out * 2 + args.out * (args.in_ // M) * N + idx_bytes + args.out * 6
    print(json.dumps({"form": "int8", "rows": args.rows, "in": args.in_, "out": args.out, "level": args.level, "out_dtype": args.dtype,
                      "ms": times, "algorithmic_bytes": alg, "kept_ops": 2.0 * args.rows * args.in_ * args.out * N / M,
                      "dense_equiv_ops": 2.0 * args.rows * args.in_ * args.out}))


def backward_case(args):
    """The backward of one layer; both products run at the dense rate, so their roofline is 2 rows in out flops
    each against the dense bf16 peak (db: the bytes of dY against the HBM peak)."""
    N, M = (int(v) for v in args.level.split(":"))
    dtype = synth.torch_dtype(args.dtype)
    layer = synth.Layer("case", args.rows, args.in_, args.out, N, M, 1, 2, 3)
    X, W, _ = synth.layer_tensors(layer, dtype, device="cuda")
    dY = synth.randn((args.rows, args.out), 4, 0.05, dtype, device="cuda")
    vals, idx = lib.elsa_nm_compress(W, N, M)
    ws = lib.alloc_workspace(lib.elsa_backward_workspace_bytes(args.rows, args.in_, args.out, N, M, lib.dtype_code(dtype)))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    out = {"form": "backward", "rows": args.rows, "in": args.in_, "out": args.out, "level": args.level, "dtype": args.dtype,
           "dense_flops_per_product": layer.dense_equiv_flops, "dY_bytes": args.rows * args.out * 2}
    for want in (("dX",), ("dW",), ("db",), ("dX", "dW", "db")):
        times = []
        for rep in range(args.reps + 1):
            flush.fill_(rep)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            lib.elsa_nm_linear_backward(dY, X, vals, idx, args.out, args.in_, N, M, want=want, workspace=ws, dev_status=status)
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        out["ms_" + "_".join(want)] = times[1:]                    # the first call also allocates its outputs' pages
    assert int(status.item()) == 0
    print(json.dumps(out))


def attention_case(args):
    """elsa_attention alone.  Its roofline is the larger of 4 tokens^2 64 FLOPs per head and image at the bf16 peak
    and the bytes of qkv in and a out at the HBM peak."""
    dtype = synth.torch_dtype(args.dtype)
    dim = 64 * args.heads
    rows = args.images * args.tokens
    qkv = synth.randn((rows, 3 * dim), 5, 1.0, dtype, device="cuda")
    a = torch.empty((rows, dim), dtype=dtype, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    times = []
    for rep in range(args.reps + 1):
        flush.fill_(rep)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        lib.elsa_attention(qkv, args.tokens, args.heads, a=a, dev_status=status)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    assert int(status.item()) == 0
    print(json.dumps({"form": "attention", "images": args.images, "tokens": args.tokens, "heads": args.heads, "dtype": args.dtype,
                      "ms": times[1:], "flops": 4.0 * args.tokens * args.tokens * 64 * args.heads * args.images,
                      "algorithmic_bytes": rows * dim * 4 * 2}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--rows", type=int, default=50432)
    ap.add_argument("--in", dest="in_", type=int, default=768)
    ap.add_argument("--out", type=int, default=3072)
    ap.add_argument("--level", default="2:8")
    ap.add_argument("--dtype", default="bf16", choices=["f16", "bf16"])
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--variant", default="auto", choices=["auto", "simt", "tc_dense", "tc_pair", "tc_sparse", "tc_sparse_pair",
                                                            "tc_sparse_ws", "tc_sparse_st"])
    ap.add_argument("--compress-table", default=None, help="workload whose weights go through elsa_vit_compress")
    ap.add_argument("--int8", action="store_true", help="the INT8 form: elsa_nm_compress_i8 once, then elsa_nm_linear_i8")
    ap.add_argument("--backward", action="store_true", help="elsa_nm_linear_backward on the layer")
    ap.add_argument("--attention", action="store_true", help="elsa_attention on --images x --tokens x --heads")
    ap.add_argument("--images", type=int, default=256)
    ap.add_argument("--tokens", type=int, default=197)
    ap.add_argument("--heads", type=int, default=12)
    args = ap.parse_args()
    if args.attention:
        return attention_case(args)
    if args.backward:
        return backward_case(args)
    if args.compress_table:
        return compress_table(args.compress_table, args.reps)
    if args.int8:
        return int8_case(args)
    N, M = (int(v) for v in args.level.split(":"))
    dtype = synth.torch_dtype(args.dtype)
    layer = synth.Layer("case", args.rows, args.in_, args.out, N, M, 1, 2, 3)
    X, W, b = synth.layer_tensors(layer, dtype, device="cuda")
    vals, idx = lib.elsa_nm_compress(W, N, M)
    Y = torch.empty((args.rows, args.out), dtype=dtype, device="cuda")
    ws = lib.alloc_workspace(lib.elsa_workspace_bytes(args.rows, args.in_, args.out, N, M, lib.dtype_code(dtype)))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    lib.elsa_set_linear_variant({"auto": lib.VARIANT_AUTO, "simt": lib.VARIANT_SIMT,
                                 "tc_dense": lib.VARIANT_TC_DENSE, "tc_pair": lib.VARIANT_TC_PAIR, "tc_sparse": lib.VARIANT_TC_SPARSE,
                                 "tc_sparse_pair": lib.VARIANT_TC_SPARSE_PAIR,
                                 "tc_sparse_ws": lib.VARIANT_TC_SPARSE_WS,
                                 "tc_sparse_st": lib.VARIANT_TC_SPARSE_ST}[args.variant])
    times = []
    for _ in range(args.reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        lib.elsa_nm_linear(X, vals, idx, b, args.out, args.in_, N, M, Y=Y, workspace=ws, dev_status=status)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    assert int(status.item()) == 0
    bits = {4: 2, 8: 3, 16: 4}[M]
    idx_bytes = 0 if N == M else args.out * (-(-(args.in_ // M * N * bits) // 32)) * 4
    alg = (args.rows * args.in_ + args.rows * args.out + args.out * (args.in_ // M) * N + args.out) * 2 + idx_bytes
    print(json.dumps({"rows": args.rows, "in": args.in_, "out": args.out, "level": args.level, "dtype": args.dtype,
                      "ms": times, "algorithmic_bytes": alg, "kept_flops": layer.kept_flops,
                      "dense_equiv_flops": layer.dense_equiv_flops}))


if __name__ == "__main__":
    main()
