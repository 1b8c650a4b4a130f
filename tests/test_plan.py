"""Host logic: the static split of a tensor list over the blocks of the persistent kernels."""
import random

import pytest


@pytest.fixture(scope="module")
def B():
    from paper_2007_05105_b200 import build
    build.build()
    from paper_2007_05105_b200 import binding
    return binding


def _check(rows, numels, unit, max_blocks):
    covered = {k: 0 for k, n in enumerate(numels) if n > 0}
    last_block = -1
    for tensor, first, length, block in rows:
        assert length > 0 and first % unit == 0
        assert first == covered[tensor], "segments of a tensor must tile it in order"
        covered[tensor] += length
        assert block >= last_block and block < max_blocks
        last_block = block
        assert length % unit == 0 or first + length == numels[tensor]
    assert covered == {k: n for k, n in enumerate(numels) if n > 0}


@pytest.mark.parametrize("unit", [4, 8])
def test_every_element_is_owned_exactly_once(B, unit):
    rng = random.Random(unit)
    for trial in range(200):
        T = rng.randint(1, 40)
        numels = [rng.choice([0, 1, 3, 7, 64, 1000, 4097, rng.randint(1, 300000)]) for _ in range(T)]
        if sum(numels) == 0:
            numels[0] = 5
        max_blocks = rng.choice([1, 2, 7, 148, 592])
        seg_cost = rng.choice([0, 4, 128, 1024])
        _check(B.plan(numels, unit, seg_cost, max_blocks), numels, unit, max_blocks)


@pytest.mark.parametrize("name,unit,S", [("resnet18", 4, 8), ("resnet50", 8, 16), ("transformer_base", 4, 32),
                                         ("decoder_24l", 8, 32), ("single_1m", 4, 4)])
def test_benchmark_workloads_are_balanced(B, name, unit, S):
    from paper_2007_05105_b200 import synthetic
    numels = synthetic.workload(name).numels
    blocks = 148 * 4
    seg_cost = max(4, 1024 // S)
    rows = B.plan(numels, unit, seg_cost, blocks)
    _check(rows, numels, unit, blocks)
    cost = {}
    for tensor, first, length, block in rows:
        cost[block] = cost.get(block, 0) + -(-length // unit) + seg_cost
    used = len(cost)
    assert used >= min(blocks, sum(numels) // unit // 512) * 0.95
    mean = sum(cost.values()) / used
    assert max(cost.values()) <= 1.05 * mean + seg_cost + 1
    # the cost model must not leave a block with (almost) nothing while others are full
    assert min(cost.values()) >= 0.5 * mean or used < blocks


def test_small_jobs_use_few_blocks(B):
    rows = B.plan([100], 4, 128, 592)
    assert len(rows) == 1 and rows[0] == (0, 0, 100, 0)
    rows = B.plan([4096], 4, 128, 592)          # 1024 units -> 2 blocks of >= 512 units
    assert {r[3] for r in rows} == {0, 1}


def test_invalid_plan_arguments(B):
    with pytest.raises(ValueError):
        B.plan([-1], 4, 0, 8)
    with pytest.raises(ValueError):
        B.plan([10], 0, 0, 8)
    with pytest.raises(ValueError):
        B.plan([10], 4, 0, 0)
