#!/usr/bin/env python
"""Benchmark of the N:M sparse-linear path on seeded synthetic ViT workloads.

One step = one pass of the whole path over the workload's layer table: elsa_vit_compress of every
layer's dense weight to its level, then elsa_vit_linears over the table (weight images the MMAs
read, then the tcgen05 GEMMs with bias; layers of a kernel family share persistent launches).  The default workload is the 48-layer DeiT-B
stack at batch 256 in bf16 with a seeded level per layer from {1:8, 2:8, 4:8, 8:8}.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line.  `value` is dense-equivalent TFLOP/s (2*R*K*O summed over layers / step
time) with inputs resident in HBM; `e2e` is the same metric through elsa_vit_linears_host with
pinned host buffers and the copies inside the timed region.  `roofline` is for the dominant
kernel (the tcgen05 GEMM), timed per launch with CUDA events in a second timed pass; the roofline
time of a layer is max(kept FLOPs / tensor peak, algorithmic bytes / HBM bandwidth).
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
With N > 1 (torchrun) every rank runs an independent replica; there is no collective on the path.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "sparse-GEMM dense-equivalent TFLOP/s over the ViT linear stack"
UNIT = "TFLOP/s"
GEMM_KERNELS = ("linear_tc_dense", "linear_tc_pair", "linear_tc_sp24", "linear_tc_sp24_pair", "linear_tc_sp24_ws", "linear_tc_sp24_st")   # forms of the tcgen05 GEMM

# dram__bytes_read.sum + dram__bytes_write.sum of each GEMM kernel's launches over ONE step of this
# benchmark, from a one-pass ncu capture of the same command (the two DRAM counters
# fit one pass, so the full-size run is captured as it is).  Valid for the kernels as captured; set an
# entry to None when its kernel changes.
MEASURED_DRAM_TRAFFIC = {
    "deit_b_stack_b256": {"linear_tc_pair": 8.773e9, "linear_tc_sp24_ws": 4.70e9, "linear_tc_sp24_pair": 3.571e9},
    "swin_b_stack_b128": {"linear_tc_pair": 10.458e9, "linear_tc_sp24_pair": 2.485e9},
}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def algorithmic_bytes(l, lib=None):
    """What the method itself must move for one layer: X in, Y out, packed values, index words, bias."""
    b = 4 if l.M == 16 else 3 if l.M == 8 else 2
    vals = l.out * (l.in_ // l.M) * l.N * 2
    idx = 0 if l.N == l.M else l.out * (-(-(l.in_ // l.M * l.N * b) // 32)) * 4
    return l.rows * l.in_ * 2 + l.rows * l.out * 2 + vals + idx + l.out * 2


def roofline_seconds(l, peaks, which="bf16_tflops"):
    t_c = l.kept_flops / (peaks[which] * 1e12)
    t_m = algorithmic_bytes(l) / (peaks["hbm_gbs"] * 1e9)
    return max(t_c, t_m), ("tensor" if t_c >= t_m else "hbm")


class ClockSampler:
    """nvidia-smi clock and throttle-reason samples while the timed region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1])); smax.append(float(parts[2])); power.append(float(parts[3]))
                except ValueError:
                    continue
                for name, v in zip(names, parts[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = [c for c, p in zip(sm, power) if p >= 0.5 * max(power)] or sm
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": max(smax), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


def max_over_ranks(ms: float, world: int, device="cuda") -> float:
    """The slowest rank's time: what a multi-GPU number is quoted on."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tflops(flops_per_rank: float, world: int, ms: float) -> float:
    """Replicas only: every rank processes the same table, the job's throughput is the sum over ranks."""
    return world * flops_per_rank / (ms * 1e-3) / 1e12


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


# ---------------------------------------------------------------------------------- CPU oracle arm

def oracle_sample(layers, dtype_name, rows_per_layer, seed=7):
    """Times the oracle, as it stands, on `rows_per_layer` seeded rows of every layer of the workload
    (weights are compressed in full).  Returns (seconds, dense-equivalent flops of the sample)."""
    import torch
    from oracle import elsa_oracle as eo
    from paper_2409_09708_b200 import synth
    dtype = synth.torch_dtype(dtype_name)
    code = eo.F16 if dtype == torch.float16 else eo.BF16
    # inputs are drawn outside the timed part
    work = []
    for l in layers:
        rows = min(rows_per_layer, l.rows)
        X = synth.bits(synth.randn((rows, l.in_), l.seed_x + seed, synth.X_STD, dtype))
        _, W, b = synth.layer_tensors(l, dtype, with_x=False)
        work.append((l, rows, X, synth.bits(W), synth.bits(b)))
    t0 = time.perf_counter()
    flops = 0.0
    for l, rows, X, W, b in work:
        vals, idx, _ = eo.nm_compress(W, l.N, l.M)
        eo.nm_linear_f64(X, vals, idx, b, l.out, l.in_, l.N, l.M, code)
        flops += 2.0 * rows * l.in_ * l.out
    return time.perf_counter() - t0, flops


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    from oracle import elsa_oracle as eo
    from paper_2409_09708_b200 import synth
    layers, dtype_name = synth.workload(args.workload)
    rows = args.oracle_rows
    for _ in range(args.warmup):
        oracle_sample(layers[:4], dtype_name, 8)
    times, flops = [], 0.0
    for _ in range(args.steps):
        t, flops = oracle_sample(layers, dtype_name, rows)
        times.append(t)
    sec = sum(times) / len(times)
    value = flops / sec / 1e12
    sample = "%d seeded rows of each of the %d layers per step (weights compressed in full)" % (rows, len(layers))
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
            "config": {"workload": args.workload, "layers": len(layers), "storage_dtype": dtype_name,
                       "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": eo.omp_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------- GPU arm

def run_ours(args):
    import torch
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the sparse-linear path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    from paper_2409_09708_b200 import build as _build
    if rank == 0:
        _build.build()
    if world > 1:
        dist.barrier()
    from paper_2409_09708_b200 import binding as lib, synth

    layers, dtype_name = synth.workload(args.workload)
    dtype = synth.torch_dtype(dtype_name)
    code = lib.dtype_code(dtype)
    peaks, peaks_kind = load_peaks()

    # ---- resident inputs (seeded, drawn on the device); every layer owns its X and Y
    dev = []
    for l in layers:
        X, W, b = synth.layer_tensors(l, dtype, device="cuda")
        vals, idx = lib.alloc_packed(l.out, l.in_, l.N, l.M, dtype)
        Y = torch.empty((l.rows, l.out), dtype=dtype, device="cuda")
        dev.append(dict(X=X, Y=Y, W=W, vals=vals, idx=idx, bias=b, N=l.N, M=l.M))
    table = lib.make_layer_table(dev)
    ws = lib.alloc_workspace(lib.elsa_vit_workspace_bytes(table, code))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    wtable = lib.make_weight_table(dev)

    def step():
        lib.elsa_vit_compress(wtable, code)
        lib.elsa_vit_linears(table, code, ws, dev_status=status)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(n_steps, profile=False):
        barrier()
        launches0 = lib.elsa_launch_count()
        if profile:
            lib.elsa_profile_start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n_steps):
            step()
        e1.record()
        barrier()
        recs = lib.elsa_profile_stop() if profile else None
        ms = max_over_ranks(e0.elapsed_time(e1), world)
        return ms, lib.elsa_launch_count() - launches0, recs

    for _ in range(args.warmup):
        step()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    total_ms, launches, _ = timed(args.steps)
    prof_ms, _, recs = timed(args.steps, profile=True)
    # a third pass with one launch per layer, only for the per-layer report
    lib.elsa_set_grouping(False)
    layer_steps = max(1, args.steps // 2)
    _, _, recs_layer = timed(layer_steps, profile=True)
    lib.elsa_set_grouping(True)
    clocks = sampler.stop() if rank == 0 else None
    assert int(status.item()) == 0, "device status %#x" % int(status.item())

    ms_per_step = total_ms / args.steps
    dense_flops = sum(l.dense_equiv_flops for l in layers)
    kept_flops = sum(l.kept_flops for l in layers)
    value = whole_job_tflops(dense_flops, world, ms_per_step)

    # ---- per-kernel accounting from the profiled pass
    per_kernel = {}
    gemm_ms = [0.0] * len(layers)
    unpack_ms = [0.0] * len(layers)
    for name, layer, ms in recs:
        k = per_kernel.setdefault(name, [0, 0.0])
        k[0] += 1
        k[1] += ms
    layer_kernel = {}                       # which GEMM kernel runs each layer (from the one-launch-per-layer pass)
    for name, layer, ms in recs_layer:
        if name in GEMM_KERNELS and layer >= 0:
            gemm_ms[layer] += ms / layer_steps
            layer_kernel[layer] = name
        if name in ("nm_unpack", "nm_to_sp24", "weight_images") and layer >= 0:
            unpack_ms[layer] += ms / layer_steps
    kernel_total = sum(v[1] for v in per_kernel.values()) or 1.0
    roof = [roofline_seconds(l, peaks) for l in layers]
    roof_sus = [roofline_seconds(l, peaks, "bf16_tflops_sustained") for l in layers]
    nominal = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}      # data-sheet figures, for context only
    roof_nom = [roofline_seconds(l, nominal) for l in layers]
    sum_roof = sum(r[0] for r in roof)
    # GEMM time per step: the shared launches of the profiled pass, as the timed region runs them
    sum_gemm = sum(per_kernel.get(k, [0, 0.0])[1] for k in GEMM_KERNELS) / args.steps * 1e-3
    share = {"tensor": sum(r[0] for r in roof if r[1] == "tensor"), "hbm": sum(r[0] for r in roof if r[1] == "hbm")}
    bound = "tensor" if share["tensor"] >= share["hbm"] else "hbm"
    frac = sum_roof / sum_gemm if sum_gemm > 0 else None
    peak = peaks["bf16_tflops"] if bound == "tensor" else peaks["hbm_gbs"]
    gemm_launches = sum(per_kernel.get(k, [0, 0.0])[0] for k in GEMM_KERNELS)
    gemm_total_ms = sum(per_kernel.get(k, [0, 0.0])[1] for k in GEMM_KERNELS)
    top_kernel = max(GEMM_KERNELS, key=lambda k: per_kernel.get(k, [0, 0.0])[1])
    top_launches = per_kernel.get(top_kernel, [0, 0.0])[0]
    roofline = {
        "kernel": top_kernel, "bound": bound, "achieved": frac * peak if frac else None, "peak": peak,
        "unit": "TFLOP/s" if bound == "tensor" else "GB/s", "frac": frac,
        # per launch, like `achieved`: the step's bytes of `kernel` over its launches per step (layers share launches)
        "traffic": (MEASURED_DRAM_TRAFFIC[args.workload][top_kernel] * args.steps / top_launches
                    if top_launches and top_kernel in MEASURED_DRAM_TRAFFIC.get(args.workload, {}) else None),
        "traffic_note": "DRAM bytes (read + written) per launch of `kernel`, whose launches carry all of its layers "
                        "(ncu, one pass, same command); traffic_algorithmic is the same layers' algorithmic bytes per launch",
        "traffic_algorithmic": (sum(algorithmic_bytes(l) for i, l in enumerate(layers) if layer_kernel.get(i) == top_kernel)
                                * args.steps / top_launches if top_launches else None),
        "peaks": peaks_kind,
        "definition": "per layer max(kept FLOPs / tensor peak, algorithmic bytes / HBM peak), summed over the "
                      "layers, divided by the summed CUDA-event durations of the GEMM launches that ran them "
                      "(layers of a kernel family share launches); achieved = frac * peak of the resource that "
                      "bounds most of the summed roofline time",
        "kept_tflops": kept_flops / sum_gemm / 1e12 if sum_gemm else None,
        "algorithmic_gbs": sum(algorithmic_bytes(l) for l in layers) / sum_gemm / 1e9 if sum_gemm else None,
        "frac_vs_sustained_peak": sum(r[0] for r in roof_sus) / sum_gemm if sum_gemm else None,
        "frac_vs_nominal_peaks": sum(r[0] for r in roof_nom) / sum_gemm if sum_gemm else None,
        "launches": gemm_launches,
        "avg_launch_ms": gemm_total_ms / max(gemm_launches, 1),
        "roofline_time_share": {k: v / sum_roof for k, v in share.items()},
    }
    # the step also compresses every weight: its own roofline is the bytes it must move (dense W in, packed
    # values and index words out) at the HBM peak
    compress_bytes = sum(l.out * l.in_ * 2 + algorithmic_bytes(l) - 2 * l.rows * (l.in_ + l.out) - l.out * 2 for l in layers)
    compress_roof = compress_bytes / (peaks["hbm_gbs"] * 1e9)
    stack_frac = (sum_roof + compress_roof) / (ms_per_step * 1e-3)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": dtype_name, "data": "synthetic",
        "config": {"workload": args.workload, "layers": len(layers), "rows": layers[0].rows,
                   "levels": sorted({"%d:%d" % (l.N, l.M) for l in layers}),
                   "l2": "inputs_exceed_l2 (every layer owns distinct X and Y; %.1f GB touched per step)"
                         % (sum(algorithmic_bytes(l) for l in layers) / 1e9),
                   "step": "elsa_vit_compress of every layer + elsa_vit_linears (layers of a kernel family share persistent "
                           "launches)", "multi_gpu": "independent replicas"},
        "actual_tflops": world * kept_flops / (ms_per_step * 1e-3) / 1e12,
        "ms_per_stack": ms_per_step,
        "stack_roofline_frac": stack_frac,
        "stack_roofline_ms": {"linears": sum_roof * 1e3, "compress": compress_roof * 1e3},
        "gpu_launches": launches,
        "roofline": roofline,
        "kernels": {k: {"launches": v[0], "ms": v[1], "share": v[1] / kernel_total} for k, v in per_kernel.items()},
        "ms_per_step_profiled": prof_ms / args.steps,
        "compress_gbs": (compress_bytes * args.steps / per_kernel["nm_compress"][1] / 1e6)
                        if per_kernel.get("nm_compress", [0, 0.0])[1] > 0 else None,
        "clocks": clocks,
    }

    # ---- per-layer report (scratch output; the committed summary is made from it)
    if rank == 0:
        rows = []
        for i, l in enumerate(layers):
            rows.append({"layer": l.name, "rows": l.rows, "in": l.in_, "out": l.out, "level": "%d:%d" % (l.N, l.M),
                         "gemm_ms": gemm_ms[i], "unpack_ms": unpack_ms[i], "roofline_ms": roof[i][0] * 1e3,
                         "bound": roof[i][1], "frac": roof[i][0] * 1e3 / gemm_ms[i] if gemm_ms[i] else None,
                         "dense_equiv_tflops": l.dense_equiv_flops / gemm_ms[i] / 1e9 if gemm_ms[i] else None,
                         "algorithmic_gbs": algorithmic_bytes(l) / gemm_ms[i] / 1e6 if gemm_ms[i] else None})
        try:
            os.makedirs(os.path.join(ROOT, "bench_out"), exist_ok=True)
            with open(os.path.join(ROOT, "bench_out", "bench_layers_%s.json" % args.workload), "w") as f:
                json.dump(rows, f, indent=1)
        except OSError:
            pass

    # ---- end to end from pinned host memory through elsa_vit_linears_host
    if not args.no_e2e:
        line["e2e"] = run_e2e(args, lib, synth, layers, dtype, code, dev, world, barrier)
    # ---- the oracle on the host cores, rank 0 at N = 1 only
    if world == 1 and not args.no_cpu_baseline:
        from oracle import elsa_oracle as eo
        sec, flops = oracle_sample(layers, dtype_name, args.oracle_rows)
        line["cpu_baseline"] = {"value": flops / sec / 1e12, "unit": UNIT, "cores": eo.omp_threads(), "kind": "oracle",
                                "sample": "%d seeded rows of each of the %d layers, weights compressed in full, "
                                          "%.1f s" % (args.oracle_rows, len(layers), sec)}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_e2e(args, lib, synth, layers, dtype, code, dev, world, barrier):
    """Same metric through the host-memory entry point: per layer H2D of W, bias and X from pinned
    memory, compress, linear, D2H of Y.  Layers of equal shape share pinned host buffers."""
    import torch
    host_x, host_y = {}, {}
    host = []
    for l, d in zip(layers, dev):
        kx, ky = (l.rows, l.in_), (l.rows, l.out)
        if kx not in host_x:
            host_x[kx] = d["X"].cpu().pin_memory()
        if ky not in host_y:
            host_y[ky] = torch.empty(ky, dtype=dtype).pin_memory()
        host.append(dict(X=host_x[kx], Y=host_y[ky], W=d["W"].cpu().pin_memory(), bias=d["bias"].cpu().pin_memory(),
                         N=l.N, M=l.M))
    table = lib.make_host_layer_table(host)
    mem = lib.alloc_workspace(lib.elsa_vit_host_device_bytes(table, code))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    h2d = sum(l.rows * l.in_ * 2 + l.out * l.in_ * 2 + l.out * 2 for l in layers)
    d2h = sum(l.rows * l.out * 2 for l in layers)
    steps = max(1, min(args.steps, args.e2e_steps))
    lib.elsa_vit_linears_host(table, code, mem, dev_status=status)       # warm-up
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        lib.elsa_vit_linears_host(table, code, mem, dev_status=status)
    e1.record()
    barrier()
    ms = max_over_ranks(e0.elapsed_time(e1) / steps, world)
    assert int(status.item()) == 0
    dense_flops = sum(l.dense_equiv_flops for l in layers)
    return {"value": whole_job_tflops(dense_flops, world, ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": ms, "steps": steps,
            "api": "elsa_vit_linears_host (pinned host buffers; layers of equal shape share them)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="deit_b_stack_b256",
                    choices=["single_layer", "deit_b_block_b64", "deit_b_stack_b256", "swin_b_stack_b128"])
    ap.add_argument("--oracle-rows", type=int, default=None,
                    help="rows per layer of the CPU-oracle sample (default 4096 for cpu_baseline, 1024 per step of --impl reference)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.oracle_rows is None:
        args.oracle_rows = 1024 if args.impl == "reference" else 4096
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
