"""Host-side logic of the N > 1 benchmark path on CPU: two gloo ranks (replicas only: the ranks exchange
nothing but the timing barrier and the max over ranks)."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port():
    """A TCP port nobody listens on right now (two test runs on one host must not meet on a fixed number)."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dev = torch.device("cpu")
    bench.dist_setup(world, dev)
    bench.barrier(world)
    # each rank measured its own time; the job's time is the slowest rank's
    ms, e2e = bench.max_over_ranks([10.0 + rank, 100.0 - rank], world, dev)
    rate = bench.aggregate_rate(64, world, ms)
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"ms": ms, "e2e": e2e, "rate": rate}, f)
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_max_time_and_aggregate(tmp_path):
    world, port = 2, free_port()
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"r{r}.json")) for r in range(world)]
    for r in res:
        assert r["ms"] == 11.0 and r["e2e"] == 100.0          # max over ranks, same on every rank
        assert r["rate"] == 2 * 64 / 0.011                    # all ranks' steps over the slowest time


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(free_port()))
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--gpus", "2"], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0 and p.stdout.strip() == ""
    env["RANK"] = "0"
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--gpus", "2", "--steps", "2"], env=env, capture_output=True, text=True, timeout=600)
    assert p.returncode == 0
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
