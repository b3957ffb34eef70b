"""Host logic of the N > 1 path of bench.py, run as two gloo ranks on the CPU.

The layer does not shard: N GPUs run N independent replicas, the job time is the slowest rank's
device time and the job value is N replicas' work over that time. The reference arm runs on rank 0
only; the other ranks leave without output.
"""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 100.0 + 25.0 * rank            # rank 1 is the slow one
        job_ms = bench.max_over_ranks(local_ms, torch.device("cpu"))
        value = bench.job_value(1e12, world, job_ms / 10)   # 10 steps
        dist.barrier()
        with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
            json.dump({"job_ms": job_ms, "value": value}, f)
    finally:
        dist.destroy_process_group()


def test_job_time_is_max_over_ranks(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    for r in res:
        assert r["job_ms"] == 125.0               # every rank sees the slowest rank's time
        # 2 replicas x 1e12 FLOP per 12.5 ms step = 160 TFLOP/s
        assert r["value"] == pytest.approx(2 * 1e12 / 12.5e-3 / 1e12)


def test_single_process_needs_no_group():
    import bench
    assert bench.max_over_ranks(3.5, torch.device("cpu")) == 3.5
    assert bench.job_value(2e12, 1, 1.0) == pytest.approx(2000.0)


def _run_reference(rank, world):
    env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
               MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", str(world),
                           "--steps", "1", "--warmup", "0", "--workload", "fp32_768x768_rho0.5",
                           "--reference-budget-s", "1"],
                          env=env, capture_output=True, text=True, timeout=300, cwd=ROOT)


def test_reference_arm_runs_on_rank0_only():
    r1 = _run_reference(1, 2)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = _run_reference(0, 2)
    assert r0.returncode == 0, r0.stderr
    lines = [l for l in r0.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["gpu_launches"] == 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"] == "fp32_768x768_rho0.5"
