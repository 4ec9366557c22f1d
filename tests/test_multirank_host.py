"""The N > 1 benchmark path on CPU: two `gloo` ranks. The hot path shards by rows with no exchange
(replicas only), so the only cross-rank logic is the aggregation of timings: max over ranks, whole-job
throughput = N x bytes / slowest rank. The reference arm must run on rank 0 alone."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, sys.argv[1])
    import torch, torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    ms_local = 2.0 if rank == 0 else 5.0          # rank 1 is the slow replica
    gbs, ms = bench.aggregate_throughput(10_000_000_000, ms_local, world)
    mx = bench.max_over_ranks([float(rank), 7.0 - rank], world)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"gbs": gbs, "ms": ms, "mx": mx, "world": world}))
    dist.destroy_process_group()
""")


def test_aggregation_over_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29541", str(script), ROOT],
                         capture_output=True, text=True, timeout=240, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    d = json.loads(line)
    assert d["world"] == 2
    assert d["ms"] == 5.0                                   # the slowest rank sets the time
    assert abs(d["gbs"] - 2 * 10.0 / 5e-3) < 1e-6           # 2 replicas x 10 GB in 5 ms = 4000 GB/s
    assert d["mx"] == [1.0, 7.0]


def test_single_rank_aggregation_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    gbs, ms = bench.aggregate_throughput(1_000_000_000, 1.0, 1)
    assert ms == 1.0 and abs(gbs - 1000.0) < 1e-9
    assert bench.max_over_ranks([3.5, 1.0], 1) == [3.5, 1.0]


def test_reference_arm_runs_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "1"], capture_output=True, text=True, timeout=120, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""          # other ranks exit 0 without work
