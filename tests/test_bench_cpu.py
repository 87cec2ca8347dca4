"""Host-side checks of bench.py that need no GPU: the max-over-ranks aggregation used for
multi-replica runs (two gloo ranks), the reference (oracle) arm's JSON line, and the workload
table."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local = 10.0 + 5.0 * rank                      # rank 1 is the slow replica
    out[rank] = bench.aggregate_max(local, dist)
    dist.destroy_process_group()


def test_replica_timing_takes_the_slowest_rank():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, 29731, out), nprocs=world, join=True)
        assert out[0] == out[1] == 15.0
    import bench
    assert bench.aggregate_max(7.5, None) == 7.5     # single process: unchanged


def test_reference_arm_prints_the_contract_line_and_only_on_rank_zero():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload",
           "config1", "--steps", "2", "--warmup", "1"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "TFLOP/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["config"]["workload"] == "config1"
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode == 0 and res.stdout.strip() == ""


def test_workload_table_matches_the_configs():
    sys.path.insert(0, ROOT)
    from paper_2406_17660_b200 import workloads
    w = workloads.get("llama7b_block")
    assert [(m, n) for _, m, n in w.shapes] == [(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)]
    assert w.T == 32768 and w.r == 1024 and w.dtype == torch.bfloat16
    assert w.flops_regular() == sum(2.0 * 1024 * 32768 * n for _, _, n in w.shapes)
    w = workloads.get("llama60m")
    assert len(w.layer_list()) == 56 and w.T == 65536 and w.r == 128 and w.K == 200
    w = workloads.get("config1")
    assert w.dtype == torch.float32 and w.alpha == 1.0 and w.K == 1
    assert workloads.get("llama1b", r=64).r == 64


def test_gpus_flag_starts_that_many_replicas_by_itself():
    """`bench.py --gpus 2` with no launcher around it re-executes itself under
    torch.distributed.run as two ranks (checked on CPU: the ranks only join a gloo group)."""
    env = {k: v for k, v in os.environ.items()
           if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--check-launch"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(l) for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and lines[0]["ranks"] == 2 and lines[0]["n_gpus"] == 2
    sys.path.insert(0, ROOT)
    import bench

    class A:
        gpus = 4
    argv = bench.replica_command(A, ["--gpus", "4", "--steps", "3"])
    assert "--nproc-per-node=4" in argv and argv[-4:] == ["--gpus", "4", "--steps", "3"]
    assert "127.0.0.1" in argv
