"""bench.py prints one JSON line with the agreed keys (small workload, few steps)."""
import json
import os
import subprocess
import sys

import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*extra, workload="single_1m", env=None):
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", workload, "--steps", "5",
                          "--warmup", "3", "--no-sweep", *extra], capture_output=True, text=True, timeout=600, cwd=ROOT,
                         env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.lstrip().startswith("{")]   # NCCL may log its version
    assert len(lines) == 1
    return json.loads(lines[0])


def test_default_line_has_the_contract_keys():
    d = _run()
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "clocks", "gpu_launches"):
        assert key in d, key
    assert d["unit"] == "GB/s" and d["n_gpus"] == 1 and d["steps"] == 5 and d["warmup"] == 3
    assert d["higher_is_better"] is True and d["scaling"] == "weak" and d["vs_baseline"] is None
    assert d["data"] == "synthetic" and d["config"]["workload"] == "single_1m" and "model" not in d["config"]
    assert d["value"] == pytest.approx(d["config"]["bytes_per_step"] / (d["ms_per_step"] * 1e-3) / 1e9, rel=1e-9)
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["frac"] == pytest.approx(r["achieved"] / r["peak"])
    assert r["achieved"] == pytest.approx(r["bytes_per_launch"] / (r["us_per_launch"] * 1e-6) / 1e9, rel=1e-9)
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and c["sample"]
    e = d["e2e"]
    assert e["h2d_bytes_per_step"] == 4 * 1048576 * 4 and e["d2h_bytes_per_step"] > 0 and 0 < e["value"] < d["value"]
    assert d["repeats"] >= 3 and d["gpu_launches"] == 2 * d["steps"] * d["repeats"]
    assert d["gpu_launches_per_block"] == 2 * d["steps"]
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    assert r["frac_of_read_probe"] > 0 and r["update_kernel"]["frac_of_rmw_probe"] > 0


def test_fused_mode_line():
    d = _run("--mode", "fused", "--no-e2e", "--no-cpu-baseline")
    assert d["config"]["mode"] == "fused" and d["gpu_launches"] == d["steps"] * d["repeats"]
    assert d["config"]["bytes_per_step"] == 1048576 * (4 * 4 + 16)


def test_both_arms_print_the_same_config():
    ours = _run("--no-e2e", "--no-cpu-baseline")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "single_1m",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    ref = json.loads(res.stdout.strip().splitlines()[-1])
    assert ref["config"] == ours["config"] and ref["metric"] == ours["metric"] and ref["unit"] == ours["unit"]


def test_sharded_mode_with_one_rank_goes_through_nccl():
    """The column-sharded sequence (reduce_sums, all-reduce of 16 bytes over NCCL, apply_sums) with a
    world of one rank: the call sequence of the multi-GPU path on the one GPU there is."""
    env = dict(os.environ, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0", MASTER_ADDR="127.0.0.1")
    env.pop("MASTER_PORT", None)
    d = _run("--mode", "sharded", workload="resnet18", env=env)
    assert d["config"]["mode"] == "sharded" and d["scaling"] == "strong" and d["n_gpus"] == 1
    assert d["sharded_check"]["ok"] is True
    assert d["gpu_launches"] == 3 * d["steps"] * d["repeats"]      # reduce, scalar, update
    assert d["value"] == pytest.approx(d["config"]["bytes_per_step"] / (d["ms_per_step"] * 1e-3) / 1e9, rel=1e-9)
