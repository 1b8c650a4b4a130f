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


def test_bench_starts_its_own_ranks(tmp_path):
    """`bench.py --gpus N` without a launcher starts N processes with RANK / LOCAL_RANK / WORLD_SIZE set."""
    sys.path.insert(0, ROOT)
    import bench
    code = ("import os; open(os.path.join(%r, 'rank' + os.environ['RANK']), 'w').write("
            "' '.join(os.environ[k] for k in ('RANK', 'LOCAL_RANK', 'WORLD_SIZE', 'MASTER_ADDR', 'MASTER_PORT')))" % str(tmp_path))
    assert bench.spawn_ranks([sys.executable, "-c", code], 3) == 0
    seen = [open(tmp_path / ("rank%d" % r)).read().split() for r in range(3)]
    assert [s[:4] for s in seen] == [[str(r), str(r), "3", "127.0.0.1"] for r in range(3)]
    assert len({s[4] for s in seen}) == 1
    assert bench.spawn_ranks([sys.executable, "-c", "import os, sys; sys.exit(int(os.environ['RANK']))"], 2) == 1


class _StubContext:
    """Stands in for the native context of one rank: hands out a recorded pair of sums and
    records what the scalar part is given."""

    def __init__(self, pair):
        self.pair = pair
        self.calls = []

    def reduce_sums(self, grads, sums, stream=None):
        import torch
        self.calls.append("reduce_sums")
        sums.copy_(torch.tensor(self.pair, dtype=torch.float64))

    def apply_sums(self, sums, sched, params, momentum, stream=None):
        self.calls.append(("apply_sums", sums.tolist()))


def _sharded_worker(rank, world, port, out_dir):
    import torch
    sys.path.insert(0, ROOT)
    from paper_2007_05105_b200 import sharded
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    recorded = [[(3.25, 0.5), (10.0, 2.0)], [(0.75, 1.5), (6.0, 1.0)]][rank]     # two steps per rank
    seen = []
    for pair in recorded:
        ctx = _StubContext(pair)
        step = sharded.ShardedAdaScale(ctx, torch.zeros(2, dtype=torch.float64))
        step.step(None, None, None, None)
        assert ctx.calls[0] == "reduce_sums" and ctx.calls[1][0] == "apply_sums" and len(ctx.calls) == 2
        seen.append(ctx.calls[1][1])
    with open(os.path.join(out_dir, "sharded%d.json" % rank), "w") as f:
        json.dump(seen, f)
    dist.destroy_process_group()


def test_sharded_step_hands_every_rank_the_same_completed_sums(tmp_path):
    mp.spawn(_sharded_worker, args=(2, _free_port(), str(tmp_path)), nprocs=2, join=True)
    got = [json.load(open(tmp_path / ("sharded%d.json" % r))) for r in range(2)]
    assert got[0] == got[1] == [[4.0, 2.0], [16.0, 3.0]]


def test_split_columns_partitions_the_tensor_list():
    sys.path.insert(0, ROOT)
    from paper_2007_05105_b200 import sharded
    numels = [1000, 7, 64, 130000, 0, 5]
    for world in (1, 2, 3, 8):
        covered = {k: [] for k in range(len(numels))}
        sizes = []
        for rank in range(world):
            pieces = sharded.split_columns(numels, rank, world)
            sizes.append(sum(n for _, _, n in pieces))
            for k, first, n in pieces:
                assert n > 0
                covered[k].append((first, n))
        assert sum(sizes) == sum(numels) and max(sizes) - min(sizes[:-1] or sizes) <= 64
        for k, spans in covered.items():     # every tensor is covered exactly once, in order
            pos = 0
            for first, n in sorted(spans):
                assert first == pos
                pos += n
            assert pos == numels[k]
