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


def _fake_stack():
    from paper_2409_09708_b200 import synth
    layers = [synth.Layer("qkv", 50432, 768, 2304, 8, 8, 0, 0, 0), synth.Layer("proj", 50432, 768, 768, 4, 8, 0, 0, 0),
              synth.Layer("fc1", 50432, 768, 3072, 2, 8, 0, 0, 0), synth.Layer("fc2", 50432, 3072, 768, 1, 8, 0, 0, 0)]
    steps = 2
    # two steps as the timed region runs them: one launch per family and step
    recs = []
    for _ in range(steps):
        recs += [("nm_compress", -1, 0.05), ("weight_images", -1, 0.04), ("linear_tc_pair", -1, 0.30),
                 ("linear_tc_sp24_ws", -1, 0.12), ("linear_tc_sp24_st", -1, 0.10)]
    # one step with one launch per layer: which family runs which layer
    recs_layer = [("linear_tc_pair", 0, 0.2), ("nm_unpack", 1, 0.01), ("linear_tc_pair", 1, 0.1),
                  ("nm_to_sp24", 2, 0.01), ("linear_tc_sp24_ws", 2, 0.12), ("nm_to_sp24", 3, 0.01),
                  ("linear_tc_sp24_st", 3, 0.10)]
    return layers, steps, recs, recs_layer


def test_account_describes_the_dominant_family_and_every_family(tmp_path):
    import bench
    peaks = {"hbm_gbs": 6500.0, "bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0}
    layers, steps, recs, recs_layer = _fake_stack()
    roof = [bench.roofline_seconds(l, peaks)[0] for l in layers]
    traffic = tmp_path / "dram_traffic.json"
    traffic.write_text(json.dumps({"captures": [
        {"workload": "fake", "kernel": "linear_tc_pair", "dram_bytes_per_step": 5.0e9, "csrc_sha256": "abc", "command": "ncu ..."}]}))
    acc, rows = bench.account(layers, peaks, "measured", recs, recs_layer, steps, 1, 0.61, "fake",
                              source_hash="abc", traffic_path=str(traffic))
    fam = acc["families"]
    assert set(fam) == {"linear_tc_pair", "linear_tc_sp24_ws", "linear_tc_sp24_st"}
    assert fam["linear_tc_pair"]["layers"] == 2 and fam["linear_tc_sp24_ws"]["layers"] == 1
    assert fam["linear_tc_pair"]["ms_per_step"] == pytest.approx(0.30)
    assert fam["linear_tc_pair"]["roofline_ms"] == pytest.approx((roof[0] + roof[1]) * 1e3)
    assert fam["linear_tc_pair"]["frac"] == pytest.approx((roof[0] + roof[1]) / 0.30e-3)
    assert fam["linear_tc_sp24_st"]["frac"] == pytest.approx(roof[3] / 0.10e-3) and fam["linear_tc_sp24_st"]["bound"] == "hbm"
    r = acc["roofline"]
    # every key of `roofline` is about the dominant family alone
    assert r["kernel"] == "linear_tc_pair" and r["launches"] == steps and r["avg_launch_ms"] == pytest.approx(0.30)
    assert r["frac"] == pytest.approx(fam["linear_tc_pair"]["frac"]) and r["bound"] == "tensor"
    assert r["achieved"] == pytest.approx(r["frac"] * 1600.0) and r["peak"] == 1600.0 and r["unit"] == "TFLOP/s"
    assert r["traffic"] == pytest.approx(5.0e9)                       # one launch per step
    assert r["traffic_algorithmic"] == pytest.approx(bench.algorithmic_bytes(layers[0]) + bench.algorithmic_bytes(layers[1]))
    assert acc["gemm_frac"] == pytest.approx(sum(roof) / 0.52e-3)
    compress_roof = acc["stack_roofline_ms"]["compress"] * 1e-3
    assert acc["stack_roofline_frac"] == pytest.approx((sum(roof) + compress_roof) / 0.61e-3)
    assert acc["kernels"]["nm_compress"]["launches"] == steps
    assert [row["kernel"] for row in rows] == ["linear_tc_pair", "linear_tc_pair", "linear_tc_sp24_ws", "linear_tc_sp24_st"]
    # a capture taken from other kernel sources is not reported
    acc2, _ = bench.account(layers, peaks, "measured", recs, recs_layer, steps, 1, 0.61, "fake",
                            source_hash="def", traffic_path=str(traffic))
    assert acc2["roofline"]["traffic"] is None and "changed" in acc2["roofline"]["traffic_note"]
    acc3, _ = bench.account(layers, peaks, "measured", recs, recs_layer, steps, 1, 0.61, "other",
                            source_hash="abc", traffic_path=str(traffic))
    assert acc3["roofline"]["traffic"] is None


def test_kernel_source_hash_follows_the_sources():
    import bench
    h = bench.kernel_source_hash()
    assert len(h) == 64 and h == bench.kernel_source_hash()
