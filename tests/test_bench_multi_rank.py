"""The N > 1 leg of bench.py is "replicas only": every rank runs the same problem on its own GPU and
the job is timed by its slowest rank.  The rank-aggregation logic is exercised here with two gloo
ranks on the CPU; the reference arm and argument handling are checked in-process."""
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
import bench  # noqa: E402


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.reduce_max_ms(10.0 + 5.0 * rank, dist, "cpu")
    q.put((rank, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_slowest_rank_times_the_job_over_gloo():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, 29611, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == {0: 15.0, 1: 15.0}
    # two replicas of 2*8192^3 flop finishing in 15 ms
    assert bench.replica_throughput(2.0 * 8192 ** 3, 2, 15.0) == pytest.approx(2 * 2.0 * 8192 ** 3 / 15e-3 / 1e12)
    assert bench.reduce_max_ms(3.0) == 3.0


def test_algorithmic_work_matches_the_derivation():
    # n = 8192, one level, rank 7, fp32 scales, block 32: 9.62e11 flop, 1334 MB moved in total
    flops, enc, gemm = bench.algorithmic_work(8192, 8192, 8192, 1, 7, 4, 32)
    assert flops == pytest.approx(9.621e11, rel=1e-3)
    assert (enc + gemm) / 1e6 == pytest.approx(1334, rel=5e-3)
    flops0, enc0, gemm0 = bench.algorithmic_work(8192, 8192, 8192, 0, 8, 4, 32)
    assert flops0 == pytest.approx(1.0995e12, rel=1e-3)
    assert (enc0 + gemm0) / 1e6 == pytest.approx(1107, rel=5e-3)


def test_combined_roofline_time_follows_the_derivation():
    # n = 8192, one level: tensor phase at the given fp8 peak plus the algorithmic bytes at the given bandwidth,
    # the same formula in every scale mode; 380.5 us at the nominal peaks (4.5 PFLOP/s, 8 TB/s)
    n, peak, bw = 8192, 3293.6, 6459.0
    for mode, sbytes, blk in (("ue8m0", 1, 32), ("fp32", 4, 32), ("fp32", 4, 128), ("fp32+tile128", 4, 128)):
        flops, enc, gemm = bench.algorithmic_work(n, n, n, 1, 7, sbytes, blk)
        want = (flops / (peak * 1e12) + (enc + gemm) / (bw * 1e9)) * 1e3
        assert bench.combined_roofline_ms(n, n, n, 1, 7, mode, blk, peak, bw) == pytest.approx(want, rel=1e-12)
    spec = bench.combined_roofline_ms(n, n, n, 1, 7, "fp32", 32, bench.SPEC_FP8_TFLOPS, bench.SPEC_HBM_GBS)
    assert spec == pytest.approx(0.3805, rel=2e-3)
    assert bench.combined_roofline_ms(n, n, n, 1, 7, "fp32", 32, peak, bw) == pytest.approx(0.4986, rel=2e-3)
    # the CUDA-core floor of the fp32-scale promotion is reported beside the roofline, never inside it
    alu = 2.0 * n * n * (n / 32) * (7 / 8) / (148 * 128 * 1.965e9) * 1e3
    assert bench.alu_floor_ms(n, n, n, 1, 7, "fp32", 32) == pytest.approx(alu, rel=1e-12)
    assert bench.alu_floor_ms(n, n, n, 1, 7, "fp32+tile128", 128) == pytest.approx(alu / 8, rel=1e-12)
    assert bench.alu_floor_ms(n, n, n, 1, 7, "ue8m0", 32) == 0.0
    pk = {"bf16_tflops": 1646.8, "hbm_gbs": 6459.0}
    fr = bench.roofline_fractions(n, n, n, 1, 7, "fp32", 32, 2.0385, pk)
    assert fr["combined_frac"] == pytest.approx(0.245, abs=2e-3) and fr["combined_frac_spec"] == pytest.approx(0.187, abs=2e-3)
    # fully overlapped phases: max(tensor time, HBM time) = 213.8 us at the nominal peaks, 292.1 us at the measured ones
    assert fr["overlap_bound_spec_ms"] == pytest.approx(0.2138, rel=2e-3)
    assert fr["overlap_bound_ms"] == pytest.approx(0.2921, rel=2e-3)


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--ref-n", "256"], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["unit"] == "TFLOP/s"
    # other ranks of a torchrun launch do no work and print nothing
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, timeout=60, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""
