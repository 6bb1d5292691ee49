"""Multi-rank plumbing of the benchmark on CPU: two gloo ranks, replicas only (max time, summed units)."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 1000.0 * (rank + 1), world)
    ret[rank] = (ms, units)
    dist.barrier()
    dist.destroy_process_group()


def test_aggregate_over_two_gloo_ranks():
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(2, 29000 + os.getpid() % 2000, ret), nprocs=2, join=True)
    assert ret[0] == ret[1] == (15.0, 3000.0)


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(7.5, 42.0, 1) == (7.5, 42.0)


def test_roofline_terms_match_the_stated_per_unit_costs():
    sys.path.insert(0, ROOT)
    import bench
    n = N = 10_000_000
    nnz, d, e = 1_000_000_000, 128, 2
    b, t, a = bench.roofline_terms(n, N, nnz, d, e)
    assert abs(b - 265.2e9) / 265.2e9 < 0.01          # bytes per half-epoch of the 10M x 10M workload
    assert abs(t - 3.31e13) / 3.31e13 < 0.01
    assert abs(a - 7.74e12) / 7.74e12 < 0.01


def test_replica_command_is_one_process_per_gpu_on_this_node():
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.replica_command(["--gpus", "4", "--steps", "2"], 4, 29555)
    assert cmd[1:3] == ["-m", "torch.distributed.run"]
    assert "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29555"
    k = cmd.index(os.path.join(ROOT, "bench.py"))
    assert cmd[k + 1:] == ["--gpus", "4", "--steps", "2"]


def test_plain_launch_with_two_gpus_spawns_two_ranks_and_prints_one_line():
    """`python bench.py --gpus 2` without a launcher's environment starts the ranks itself.  Run on the reference arm
    (CPU only): rank 0 alone works and prints, the other rank exits 0, the launcher passes the exit code on."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference",
                          "--workload", "small", "--steps", "1", "--warmup", "0"], env=env, capture_output=True,
                         text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["value"] > 0
