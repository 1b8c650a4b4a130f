"""N > 1 path of bench.py on CPU: two gloo ranks, timing reduction and rank-0-only reference arm."""
import json
import os
import socket
import subprocess
import sys

import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    w, r, local = bench.dist_setup(world)
    assert (w, r, local) == (world, rank, rank)
    bench.barrier(w)
    local_ms = 2.0 if rank == 0 else 5.0          # rank 1 is the slow replica
    ms, value = bench.whole_job_value(local_ms, 1_000_000_000, w)
    with open(os.path.join(out_dir, "r%d.json" % rank), "w") as f:
        json.dump({"ms": ms, "value": value}, f)
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_summed_rate(tmp_path):
    mp.spawn(_worker, args=(2, _free_port(), str(tmp_path)), nprocs=2, join=True)
    for rank in range(2):
        got = json.load(open(tmp_path / ("r%d.json" % rank)))
        assert got["ms"] == 5.0                                  # max over ranks
        assert abs(got["value"] - 2 * 1e9 / 5e-3 / 1e9) < 1e-9   # both replicas at the slowest pace


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--workload", "single_1m", "--steps", "1", "--warmup", "0"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0 and res.stdout.strip() == ""
    env["RANK"] = "0"
    env["LOCAL_RANK"] = "0"
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--workload", "single_1m", "--steps", "2", "--warmup", "1"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["value"] > 0 and line["e2e"]["h2d_bytes_per_step"] == 0 and line["n_gpus"] == 2


def _exchange_worker(rank, world, port, out_dir):
    import torch
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # the one exchange of the column-sharded path: each rank's (D, N) pair, summed over ranks
    sums = torch.tensor([1.5 + rank, 0.25 * (rank + 1)], dtype=torch.float64)
    dist.all_reduce(sums, op=dist.ReduceOp.SUM)
    with open(os.path.join(out_dir, "s%d.json" % rank), "w") as f:
        json.dump(sums.tolist(), f)
    dist.destroy_process_group()


def test_sharded_exchange_gives_every_rank_the_same_sums(tmp_path):
    mp.spawn(_exchange_worker, args=(2, _free_port(), str(tmp_path)), nprocs=2, join=True)
    got = [json.load(open(tmp_path / ("s%d.json" % r))) for r in range(2)]
    assert got[0] == got[1] == [1.5 + 2.5, 0.25 + 0.5]
