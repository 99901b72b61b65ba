"""Host logic of bench.py: byte accounting and the multi-replica aggregation
(two gloo ranks on CPU stand in for two GPUs running independent replicas)."""
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


def test_algorithmic_bytes_match_the_closed_form():
    # n * N * (6 + 8/B); config 3: N=8, n=8192*5376, B=256 -> 2124.9 MB
    n, N, B = 8192 * 5376, 8, 256
    assert bench.ring_schedule_bytes(N, n, B) == n * N * (6 + 8 / B)
    assert round(bench.ring_schedule_bytes(N, n, B) / 1e6, 1) == 2124.9
    assert bench.chain_fused_bytes(N, n) == 4 * n * N
    total = (bench.launch_bytes("quantize_blocks", N, n, B)
             + (N - 1) * bench.launch_bytes("rs_step_dequant_add_requant", N, n, B)
             + bench.launch_bytes("ag_dequant", N, n, B))
    assert total == bench.ring_schedule_bytes(N, n, B)


def test_aggregate_value_is_whole_job():
    # 2 replicas, each reducing 1e9 bytes in 1 ms -> 2000 GB/s
    assert bench.aggregate_value(1e9, 1.0, 2) == pytest.approx(2000.0)


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 1.0 + 2.0 * rank                      # rank 1 is the slow replica
    got = bench.max_over_ranks(ms, world, torch.device("cpu"))
    dist.barrier()
    q.put((rank, got))
    dist.destroy_process_group()


def test_max_over_ranks_two_gloo_processes():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == {0: 3.0, 1: 3.0}


def test_reference_arm_prints_one_line_and_other_ranks_stay_silent():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "3",
                          "--warmup", "3", "--workload", "C1"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env["RANK"] = "0"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "3",
                          "--warmup", "3", "--workload", "C1"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "GB/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_sweep_summary_from_a_results_file(tmp_path):
    """The sweep's markdown summary is plain host code: feed it two fabricated result lines."""
    from paper_2506_17615_b200 import sweep
    rows = []
    for nbytes, frac in ((1 << 20, 0.4), (1 << 26, 0.96)):
        leg = {"ms": 1.0, "gbs_in": 1000.0, "frac": frac}
        rows.append({"nranks": 8, "bytes_per_rank": nbytes, "block": 256, "dist": "normal", "iters": 5, "sets": 2,
                     "pipelined": leg, "by_steps": dict(leg, frac=frac * 0.75), "bf16_sim": leg,
                     "peak_gbs": 6534.1, "peak_source": "measured"})
    path = tmp_path / "sweep.jsonl"
    path.write_text("\n".join(json.dumps(r) for r in rows) + "\n")
    text = sweep.summarize(str(path))
    assert "| 8 | 256 | 1 MB | 1000 (0.400)" in text and "| 8 | 256 | 64 MB | 1000 (0.960)" in text
    assert "All 1 points with at least 64 MB per rank: single launch 0.960 - 0.960" in text


@pytest.mark.gpu
def test_bench_line_on_the_gpu_is_consistent():
    """One short run on the smallest config: the line carries the contract's keys, each roofline fraction
    is its bytes over its time over its peak, the parity verdict is bit-exact, e2e moved the bytes it names."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "C1", "--steps", "5",
                          "--min-seconds", "0.02"], capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "e2e", "gpu_launches", "clocks", "roofline", "cpu_baseline"):
        assert key in line, key
    n, count, block = 4, 65536, 256
    assert line["config"]["workload"].startswith("C1") and line["gpu_launches"] == 5
    r = line["roofline"]
    assert r["bytes_per_launch"] == 4 * count * n and r["kernel"] == "chain_fused_kernel"
    assert r["achieved"] == pytest.approx(r["bytes_per_launch"] / (line["ms_per_step"] * 1e-3) / 1e9, rel=1e-9)
    assert r["frac"] == pytest.approx(r["achieved"] / r["peak"], rel=1e-9)
    assert line["value"] == pytest.approx(2 * count * n / (line["ms_per_step"] * 1e-3) / 1e9, rel=1e-9)
    b = line["by_steps"]["roofline"]
    assert b["bytes_per_launch"] == count * n * (6 + 8 / block)
    assert b["frac"] == pytest.approx(b["bytes_per_launch"] / (line["by_steps"]["ms_per_step"] * 1e-3) / 1e9 / b["peak"], rel=1e-9)
    assert line["parity"]["verdict"] == "bit-exact" and line["parity"]["checked_words"] == n * count
    assert line["e2e"]["h2d_bytes_per_step"] == 2 * count * n == line["e2e"]["d2h_bytes_per_step"]
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1


@pytest.mark.gpu
def test_sweep_point_runs_and_accounts_bytes_per_schedule():
    """One small point of the message-size sweep: three schedules timed, each fraction against its own bytes."""
    from paper_2506_17615_b200 import sweep
    rec = sweep.run_point(4, 1 << 20, 256, "uniform", 6534.1)
    n = (1 << 20) // 2
    for key, nbytes in (("pipelined", 4 * n * 4), ("by_steps", n * 4 * (6 + 8 / 256)), ("bf16_sim", n * (8 * 4 - 4))):
        leg = rec[key]
        assert leg["ms"] > 0
        assert leg["frac"] == pytest.approx(nbytes / (leg["ms"] * 1e-3) / 1e9 / 6534.1, rel=1e-9)
        assert leg["gbs_in"] == pytest.approx(2 * n * 4 / (leg["ms"] * 1e-3) / 1e9, rel=1e-9)
    assert sweep.run_point(3, 1 << 20, 256, "uniform", 6534.1) is None       # not divisible by nranks * block
