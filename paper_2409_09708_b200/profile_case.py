"""Runs one N:M linear layer a few times through the C ABI: a small, bounded case for profilers.

    python -m paper_2409_09708_b200.profile_case --rows 50432 --in 768 --out 3072 --level 2:8 \
        --dtype bf16 --reps 3

Prints one JSON line with the CUDA-event time of each repetition (compress once, then `reps`
calls of elsa_nm_linear), the layer's algorithmic bytes and kept FLOPs.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as lib
from . import synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--rows", type=int, default=50432)
    ap.add_argument("--in", dest="in_", type=int, default=768)
    ap.add_argument("--out", type=int, default=3072)
    ap.add_argument("--level", default="2:8")
    ap.add_argument("--dtype", default="bf16", choices=["f16", "bf16"])
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--variant", default="auto", choices=["auto", "simt", "tc_dense", "tc_pair", "tc_sparse", "tc_sparse_pair",
                                                            "tc_sparse_ws"])
    args = ap.parse_args()
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
                                 "tc_sparse_ws": lib.VARIANT_TC_SPARSE_WS}[args.variant])
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
