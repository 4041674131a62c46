"""Host-side checks of bench.py that need no GPU: the multi-rank aggregation (world size 2 over
gloo), the reference arm's rank handling, and the roofline arithmetic."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms = bench.max_over_ranks(1.0 + rank, world, device="cpu")        # ranks report 1 ms and 2 ms
    out.put((rank, ms, bench.whole_job_tflops(1e12, world, ms)))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_summed_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, 29517, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, tflops in got:
        assert ms == 2.0                                 # max over ranks
        assert tflops == pytest.approx(2 * 1e12 / 2e-3 / 1e12)   # two replicas' work over the slowest time


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "1", "--oracle-rows", "4"], env=env, capture_output=True, text=True,
                       timeout=600)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "1", "--oracle-rows", "4", "--workload", "deit_b_block_b64"],
                       env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["gpu_launches"] == 0


def test_roofline_arithmetic():
    import bench
    from paper_2409_09708_b200 import synth
    peaks = {"hbm_gbs": 6500.0, "bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0}
    fc1 = synth.Layer("fc1", 50432, 768, 3072, 2, 8, 0, 0, 0)
    nbytes = bench.algorithmic_bytes(fc1)
    # X + Y + kept values + 3-bit indices (rows word-aligned) + bias
    assert nbytes == 50432 * 768 * 2 + 50432 * 3072 * 2 + 3072 * 192 * 2 + 3072 * 18 * 4 + 3072 * 2
    t, bound = bench.roofline_seconds(fc1, peaks)
    assert bound == "hbm" and t == pytest.approx(nbytes / 6500e9)
    dense = synth.Layer("fc1", 50432, 768, 3072, 8, 8, 0, 0, 0)
    t, bound = bench.roofline_seconds(dense, peaks)
    assert bound == "tensor" and t == pytest.approx(2 * 50432 * 768 * 3072 / 1600e12)
