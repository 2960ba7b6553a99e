"""The multi-rank leg of the benchmark on CPU: two gloo ranks, each an independent replica.  Checks
the reduction the bench applies (max of the ranks' device times, whole-job throughput) and that only
rank 0 of the oracle arm does work."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    from paper_2505_05086_b200.replicas import job_throughput, max_over_ranks
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 10.0 if rank == 0 else 25.0          # rank 1 is the slow replica
    value, ms = job_throughput(units_per_rank=100.0, ms_local=ms_local)
    lo = max_over_ranks(-float(rank))
    dist.barrier()
    dist.destroy_process_group()
    with open(out + f".{rank}", "w") as f:
        json.dump({"value": value, "ms": ms, "lo": lo}, f)


def test_two_gloo_ranks_reduce_to_the_slowest_replica(tmp_path):
    world, port = 2, 29000 + os.getpid() % 2000
    out = str(tmp_path / "r")
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    res = [json.load(open(out + f".{r}")) for r in range(world)]
    for r in res:
        assert r["ms"] == 25.0                       # every rank sees the slowest rank's time
        assert abs(r["value"] - 2 * 100.0 / 25e-3) < 1e-9   # units of both replicas over that time
        assert r["lo"] == 0.0


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    from paper_2505_05086_b200.replicas import job_throughput
    value, ms = job_throughput(50.0, 5.0)
    assert ms == 5.0 and abs(value - 1e4) < 1e-9


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "0",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "0",
                        "--steps", "2", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0
