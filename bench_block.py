"""Timing of the chained transformer block (elsa_vit_block): the twelve blocks of DeiT-B at batch 256, each
with the levels the stack workload gives its four linears, chained (a block's y is the next block's x).

    python bench_block.py [--blocks 12] [--batch 256] [--reps 5] [--out bench_out/block.json]
    python bench_block.py --compare          # dense 4:4 against N:4 configurations at the paper's operating points
    python bench_block.py --swin             # the 24 blocks of Swin-B at batch 128, stage by stage
    python bench_block.py --latency-cost     # F(alpha) with measured latencies as the cost table (Sec. 3.2)

Two timings: with the library's multi-head self-attention (elsa_vit_encoder: the encoder blocks of DeiT-B as
they run, without patch embedding, final norm and classifier head), and with the stand-in a = V in its place (the linear and
elementwise path alone: LayerNorms, the four N:M linears, GELU, residuals).
CUDA-event times of `reps` passes over all blocks (activations of one block alone exceed L2), one more pass with
per-launch events for the split by kernel family, and the roofline of the pass: per linear the larger of kept
FLOPs / bf16 peak and algorithmic bytes / HBM peak, plus the elementwise stages' bytes (LayerNorm in and out
twice, one residual operand per add; the copy in and out for the stand-in) / HBM peak, plus, with attention, the
larger of its 4 tokens^2 d FLOPs per head and image / bf16 peak and its bytes (qkv in, a out) / HBM peak.

--compare runs the encoder three times: every linear dense (4:4), and under two N:4 configurations {1:4, 2:4, 4:4}
drawn by the library's two-step sampler (Alg. 3) at 7.0 and 6.0 whole-model GMACs per image, the two operating
points Table 1 lists for ELSA-DeiT-B-N:4 (the paper expects up to 2.9x at 6.0 G from a cited accelerator's
MAC-proportional model; it measures no speed itself).  The searched configurations themselves need the trained
supernet; these are draws from the same search space at the same cost.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2409_09708_b200 import binding as lib
from paper_2409_09708_b200 import synth


def run(blocks=12, batch=256, reps=5, peaks=None, peaks_kind=None, roofline_seconds=None, levels=None, stand_in=True):
    """Times the chained blocks; returns the record main() prints.  peaks / roofline_seconds: bench.py's (passed in
    by bench.py itself when it calls this; looked up there otherwise).  levels: one (N, M) per linear in the order
    of the stack workload, or None for that workload's own seeded draw."""
    if peaks is None:
        import bench
        peaks, peaks_kind = bench.load_peaks()
        roofline_seconds = bench.roofline_seconds
    args = argparse.Namespace(blocks=blocks, batch=batch, reps=reps)
    dtype = torch.bfloat16
    dim, mlp = 768, 3072
    layers = synth.deit_b_stack(args.batch)[:4 * args.blocks]
    if levels is not None:
        import dataclasses
        layers = [dataclasses.replace(l, N=n, M=m) for l, (n, m) in zip(layers, levels)]
    rows = layers[0].rows

    blocks = []
    for b in range(args.blocks):
        lin = {}
        for l in layers[4 * b:4 * b + 4]:
            _, W, bias = synth.layer_tensors(l, dtype, "cuda", with_x=False)
            vals, idx = lib.elsa_nm_compress(W, l.N, l.M)
            lin[l.name.split(".")[1]] = (vals, idx, bias, l.N, l.M)
        ln = [synth.randn((dim,), 9000 + 4 * b + i, 0.1, dtype, "cuda") + (1.0 if i % 2 == 0 else 0.0) for i in range(4)]
        ln = [t.to(dtype) for t in ln]
        blocks.append(lib.make_block_weights(ln[0], ln[1], ln[2], ln[3], lin))
    scratch_bytes = max(lib.elsa_vit_block_scratch_bytes(rows, dim, mlp, w, lib.BF16)[0] for w, _ in blocks)
    scratch = lib.alloc_workspace(scratch_bytes)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    x = [synth.randn((rows, dim), 77, 1.0, dtype, "cuda"), torch.empty((rows, dim), dtype=dtype, device="cuda")]

    tokens, heads = 197, 12
    x0 = x[0].clone()
    lin_roof = sum(roofline_seconds(l, peaks)[0] for l in layers)
    hbm = peaks["hbm_gbs"] * 1e9
    attn_roof = max(4.0 * tokens * tokens * 64 * heads * args.batch / (peaks["bf16_tflops"] * 1e12), rows * dim * 4 * 2 / hbm)

    table = lib.make_encoder_table([w for w, _ in blocks])
    enc_scratch = lib.alloc_workspace(int(lib._encoder_scratch(args.batch, tokens, dim, mlp, table, len(blocks), lib.BF16)))

    def measure(attention):
        def one_pass():
            if attention:      # one call for the whole encoder
                lib.elsa_vit_encoder(x[0], tokens, heads, mlp, table, y=x[args.blocks & 1], scratch=enc_scratch, dev_status=status)
                return
            for b, (w, _) in enumerate(blocks):
                lib.elsa_vit_block(x[b & 1], mlp, w, y=x[(b + 1) & 1], scratch=scratch, dev_status=status)

        for _ in range(3):
            x[0].copy_(x0)
            one_pass()
        times = []
        for _ in range(args.reps):
            x[0].copy_(x0)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            one_pass()
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        assert int(status.item()) == 0, "device status %#x" % int(status.item())
        assert torch.isfinite(x[args.blocks & 1].float()).all()
        x[0].copy_(x0)
        lib.elsa_profile_start()
        one_pass()
        families = {}
        launch_list = lib.elsa_profile_stop()
        for kernel, _, ms in launch_list:
            f = families.setdefault(kernel, {"launches": 0, "ms": 0.0})
            f["launches"] += 1
            f["ms"] += ms
        # elementwise stages per block: LayerNorm twice (in + out), two residual operands; the stand-in adds its copy
        elementwise_bytes = args.blocks * (6 if attention else 8) * rows * dim * 2
        roof_ms = (lin_roof + elementwise_bytes / hbm + (args.blocks * attn_roof if attention else 0.0)) * 1e3
        ms = statistics.median(times)
        return {"ms_per_pass": ms, "ms_min": min(times), "ms_max": max(times), "images_per_s": args.batch / ms * 1e3,
                "roofline_ms": roof_ms, "roofline_frac": roof_ms / ms, "families_profiled_pass": families,
                "first_block_launches": [[k, round(t, 4)] for k, _, t in launch_list[:len(launch_list) // args.blocks + 2]]}

    with_attention = measure(True)
    stand_in = measure(False) if stand_in else None
    rec = {"workload": "deit_b_blocks_b%d" % args.batch, "blocks": args.blocks, "rows": rows, "dtype": "bf16",
           "peaks": peaks_kind, "linears_roofline_ms": lin_roof * 1e3, "attention_roofline_ms_per_block": attn_roof * 1e3,
           "encoder_blocks_with_attention": with_attention,
           "linear_and_elementwise_path_only_standin_a_eq_v": stand_in,
           "levels": ["%d:%d" % (l.N, l.M) for l in layers]}
    return rec


def run_swin(batch=128, reps=5, pack=1):
    """The 24 blocks of Swin-B (elsa_swin_block), chained inside each stage, with the levels of the Swin-B stack
    workload; window 7, every second block shifted by 3 (none in the last stage, whose grid is one window).  Patch
    embedding, the patch-merging linears between the stages, final norm and head are not part of it: each stage
    starts from a seeded input of its own shape.  pack: windows per attention item."""
    import bench
    peaks, peaks_kind = bench.load_peaks()
    hbm = peaks["hbm_gbs"] * 1e9
    dtype = torch.bfloat16
    layers = synth.swin_b_stack(batch)
    grids = (56, 28, 14, 7)
    heads_of = (4, 8, 16, 32)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stages, li = [], 0
    for st, (dim, depth, g) in enumerate(zip(synth.SWIN_B_DIMS, synth.SWIN_B_DEPTHS, grids)):
        rows, heads, mlp, T = batch * g * g, heads_of[st], 4 * dim, 49
        blocks = []
        for b in range(depth):
            lin = {}
            for l in layers[li:li + 4]:
                _, W, bias = synth.layer_tensors(l, dtype, "cuda", with_x=False)
                vals, idx = lib.elsa_nm_compress(W, l.N, l.M)
                lin[l.name.split(".")[2]] = (vals, idx, bias, l.N, l.M)
            li += 4
            ln = [(synth.randn((dim,), 9500 + 4 * li + i, 0.1, dtype, "cuda") + (1.0 if i % 2 == 0 else 0.0)).to(dtype) for i in range(4)]
            shift = 3 if (b % 2 == 1 and g > 7) else 0
            rel = lib.elsa_swin_pack_bias(torch.randn((heads, T, T), generator=torch.Generator().manual_seed(9700 + li)) * 0.5,
                                          7, pack=pack).cuda()
            mask = lib.elsa_swin_mask(g, g, 7, shift, pack=pack).cuda() if shift else None
            blocks.append((lib.make_block_weights(ln[0], ln[1], ln[2], ln[3], lin), shift, rel, mask))
        scratch = lib.alloc_workspace(max(lib.elsa_vit_block_scratch_bytes(rows, dim, mlp, w[0], lib.BF16)[0] for w, _, _, _ in blocks))
        x = [synth.randn((rows, dim), 78 + st, 1.0, dtype, "cuda"), torch.empty((rows, dim), dtype=dtype, device="cuda")]
        stages.append(dict(dim=dim, g=g, heads=heads, mlp=mlp, rows=rows, blocks=blocks, scratch=scratch, x=x, x0=x[0].clone()))

    def one_pass():
        for s in stages:
            for b, (w, shift, rel, mask) in enumerate(s["blocks"]):
                lib.elsa_swin_block(s["x"][b & 1], s["g"], s["g"], 7, shift, s["heads"], s["mlp"], w[0], rel, mask,
                                    y=s["x"][(b + 1) & 1], scratch=s["scratch"], dev_status=status, pack=pack)

    def reset():
        for s in stages:
            s["x"][0].copy_(s["x0"])

    for _ in range(3):
        reset()
        one_pass()
    times = []
    for _ in range(reps):
        reset()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        one_pass()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    assert int(status.item()) == 0, "device status %#x" % int(status.item())
    for s in stages:
        assert torch.isfinite(s["x"][len(s["blocks"]) & 1].float()).all()
    reset()
    lib.elsa_profile_start()
    one_pass()
    families = {}
    for kernel, _, ms in lib.elsa_profile_stop():
        f = families.setdefault(kernel, {"launches": 0, "ms": 0.0})
        f["launches"] += 1
        f["ms"] += ms
    lin_roof = sum(bench.roofline_seconds(l, peaks)[0] for l in layers)
    # per block: LayerNorm in and out twice, two residual operands, attention's qkv in and a out
    other_bytes = sum(len(s["blocks"]) * (6 + 4) * s["rows"] * s["dim"] * 2 for s in stages)
    roof_ms = (lin_roof + other_bytes / hbm) * 1e3
    ms = statistics.median(times)
    return {"workload": "swin_b_blocks_b%d" % batch, "blocks": 24, "dtype": "bf16", "peaks": peaks_kind, "windows_per_attention_item": pack,
            "note": "blocks chained inside each stage; no patch embedding, patch merging, final norm or head",
            "ms_per_pass": ms, "ms_min": min(times), "ms_max": max(times), "images_per_s": batch / ms * 1e3,
            "roofline_ms": roof_ms, "roofline_frac": roof_ms / ms, "linears_roofline_ms": lin_roof * 1e3,
            "families_profiled_pass": families, "levels": ["%d:%d" % (l.N, l.M) for l in layers]}


def latency_cost(args):
    """F(alpha) of Sec. 3.2 with measured latency in place of MACs: time each DeiT-B linear shape at each level of the
    N:4 space through elsa_nm_linear, hand the table (in microseconds) to the library's cost model and two-step
    sampler, and compare the cost it predicts for the drawn configurations with the encoder's measured time."""
    import numpy as np
    dtype = torch.bfloat16
    rows = args.batch * 197
    shapes = {"qkv": (768, 2304), "proj": (768, 768), "fc1": (768, 3072), "fc2": (3072, 768)}
    levels = [(1, 4), (2, 4), (4, 4)]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    table = {}
    for name, (k, o) in shapes.items():
        X = synth.randn((rows, k), 5, 1.0, dtype, "cuda")
        W = synth.randn((o, k), 6, synth.W_STD, dtype, "cuda")
        b = synth.randn((o,), 7, synth.B_STD, dtype, "cuda")
        Y = torch.empty((rows, o), dtype=dtype, device="cuda")
        row = []
        for N, M in levels:
            vals, idx = lib.elsa_nm_compress(W, N, M)
            ws = lib.alloc_workspace(lib.elsa_workspace_bytes(rows, k, o, N, M, lib.BF16))
            # sustained latency: many calls back to back between one pair of events, as the layer runs inside a model
            # (a single cold call runs at a clock the power cap does not allow for long)
            calls = 40
            for _ in range(10):
                lib.elsa_nm_linear(X, vals, idx, b, o, k, N, M, Y=Y, workspace=ws, dev_status=status)
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(calls):
                lib.elsa_nm_linear(X, vals, idx, b, o, k, N, M, Y=Y, workspace=ws, dev_status=status)
            e1.record()
            torch.cuda.synchronize()
            row.append(e0.elapsed_time(e1) * 1e3 / calls)
        table[name] = row
        del X, Y
    order = ["qkv", "proj", "fc1", "fc2"] * args.blocks
    cost = [table[n] for n in order]
    dense = run(args.blocks, args.batch, args.reps, levels=[(4, 4)] * len(order), stand_in=False)["encoder_blocks_with_attention"]
    # what is not a pruned linear, calibrated at the dense end: the dense encoder's time minus its linears' table cost
    # (attention, the row-wise kernels, and the gaps between dependent launches that a per-kernel sum does not see)
    fixed = dense["ms_per_pass"] * 1e3 - sum(c[2] for c in cost)
    other_kernels = sum(v["ms"] for k, v in dense["families_profiled_pass"].items() if k in ("attention", "block_rowwise")) * 1e3
    lower = lib.elsa_config_cost(cost, [0] * len(cost), fixed)
    upper = lib.elsa_config_cost(cost, [2] * len(cost), fixed)
    n_int = 8
    out = []
    rng = np.random.default_rng(0)
    for interval in (1, 4, 6):
        u = [(interval + 0.5) / n_int] + [float(v) for v in rng.random(len(cost))]
        choice, got_interval = lib.elsa_two_step_sample(cost, [[1.0, 1.0, 1.0]] * len(cost), fixed, upper, n_int, 1.0, u)
        picked = [levels[c] for c in choice]
        predicted = lib.elsa_config_cost(cost, choice, fixed)
        m = run(args.blocks, args.batch, args.reps, levels=picked, stand_in=False)["encoder_blocks_with_attention"]
        out.append({"interval": got_interval, "interval_bounds_us": [lower + (upper - lower) * got_interval / n_int,
                                                                     lower + (upper - lower) * (got_interval + 1) / n_int],
                    "levels": ["%d:%d" % lv for lv in picked], "predicted_us": predicted, "measured_us": m["ms_per_pass"] * 1e3,
                    "measured_over_predicted": m["ms_per_pass"] * 1e3 / predicted})
    return {"workload": "deit_b_encoder_blocks_b%d" % args.batch,
            "cost_unit": "microseconds per call of elsa_nm_linear, 40 calls back to back",
            "levels": ["%d:%d" % lv for lv in levels], "latency_table_us": table, "fixed_cost_us": fixed,
            "attention_and_rowwise_kernels_us": other_kernels,
            "dense_encoder_us": dense["ms_per_pass"] * 1e3, "cost_range_us": [lower, upper], "draws": out}


def compare(args):
    import bench
    layers = synth.deit_b_stack(args.batch)[:4 * args.blocks]
    runs = [("dense 4:4", [(4, 4)] * len(layers), None)]
    for gmacs in (7.0, 6.0):
        picked, cost = bench.sampled_levels(lib, layers, gmacs)
        runs.append(("N:4 sampled at %.1f GMACs" % gmacs, picked, cost))
    out = []
    for name, levels, cost in runs:
        r = run(args.blocks, args.batch, args.reps, levels=levels, stand_in=False)["encoder_blocks_with_attention"]
        kept = sum(n / m for n, m in levels) / len(levels)
        out.append({"configuration": name, "whole_model_gmacs_per_image": cost, "mean_linear_density": kept,
                    "levels": ["%d:%d" % lv for lv in levels], "ms_per_pass": r["ms_per_pass"], "ms_min": r["ms_min"],
                    "images_per_s": r["images_per_s"], "roofline_frac": r["roofline_frac"],
                    "families_ms": {k: round(v["ms"], 3) for k, v in r["families_profiled_pass"].items()}})
    for o in out:
        o["speedup_over_dense"] = out[0]["ms_per_pass"] / o["ms_per_pass"]
    return {"workload": "deit_b_encoder_blocks_b%d" % args.batch, "blocks": args.blocks, "dtype": "bf16",
            "note": "encoder blocks only (no patch embedding, final norm or head); configurations are draws of the "
                    "two-step sampler from the N:4 space at the paper's operating points, not the paper's searched ones",
            "runs": out}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--blocks", type=int, default=12)
    ap.add_argument("--batch", type=int, default=256)
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--out", default="bench_out/block.json")
    ap.add_argument("--compare", action="store_true", help="dense 4:4 against sampled N:4 configurations at 7.0 and 6.0 GMACs")
    ap.add_argument("--swin", action="store_true", help="the 24 blocks of Swin-B at batch 128")
    ap.add_argument("--latency-cost", action="store_true", help="measured latencies as the cost table of F(alpha)")
    ap.add_argument("--pack", type=int, default=1, help="--swin: windows per attention item (1 or 2)")
    args = ap.parse_args()
    if args.latency_cost:
        rec = latency_cost(args)
    elif args.swin:
        rec = run_swin(128, args.reps, args.pack)
    elif args.compare:
        rec = compare(args)
    else:
        rec = run(args.blocks, args.batch, args.reps)
    os.makedirs(os.path.dirname(args.out) or ".", exist_ok=True)
    json.dump(rec, open(args.out, "w"), indent=1)
    print(json.dumps(rec))


if __name__ == "__main__":
    main()
