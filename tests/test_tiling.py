"""Host logic: how the reduce kernel tiles a tensor list (tile t goes to block t mod grid)."""
import random

import pytest


@pytest.fixture(scope="module")
def B():
    from paper_2007_05105_b200 import build
    build.build()
    from paper_2007_05105_b200 import binding
    return binding


def _cover(numels, aligned, tp, sp, cols, scalar_tile=2048):
    """Replays the kernel's walk over the tiles and returns, per tensor, the covered elements."""
    T = len(numels)
    covered = [[] for _ in range(T)]
    k = 0
    for t in range(tp[T]):
        while t >= tp[k + 1]:
            k += 1
        c0 = (t - tp[k]) * cols
        n8 = numels[k] & ~7
        covered[k].append((c0, min(cols, n8 - c0)))
    k = 0
    for t in range(sp[T]):
        while t >= sp[k + 1]:
            k += 1
        start = (numels[k] & ~7) if aligned[k] else 0
        first = start + (t - sp[k]) * scalar_tile
        covered[k].append((first, min(scalar_tile, numels[k] - first)))
    return covered


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_every_element_is_covered_exactly_once(B, dtype):
    rng = random.Random(7)
    for trial in range(150):
        T = rng.randint(1, 30)
        numels = [rng.choice([0, 1, 7, 8, 9, 64, 1000, 4097, rng.randint(1, 200000)]) for _ in range(T)]
        aligned = [rng.random() < 0.8 for _ in range(T)]
        S = rng.choice([1, 2, 3, 4, 8, 16, 17, 32, 100])
        tp, sp, cols, rows = B.tiling(numels, S, dtype, aligned, rng.choice([1, 8, 296]))
        assert rows == min(S, 8) and cols % 256 == 0
        esz = 2 if dtype == "bf16" else 4
        assert rows * cols * esz <= 32 * 1024 and cols // 256 * esz in (8, 16, 32)
        for k, spans in enumerate(_cover(numels, aligned, tp, sp, cols)):
            spans.sort()
            pos = 0
            for first, length in spans:
                assert first == pos and length > 0
                pos += length
            assert pos == numels[k]
            if not aligned[k]:
                assert tp[k + 1] == tp[k]


@pytest.mark.parametrize("name,S,dtype,expect_cols", [("resnet18", 8, "f32", 1024), ("resnet50", 16, "bf16", 2048),
                                                      ("transformer_base", 32, "f32", 1024),
                                                      ("decoder_24l", 32, "bf16", 2048), ("single_1m", 4, "f32", 1024)])
def test_benchmark_workloads(B, name, S, dtype, expect_cols):
    from paper_2007_05105_b200 import synthetic
    numels = synthetic.workload(name).numels
    tp, sp, cols, rows = B.tiling(numels, S, dtype, None, 296)
    assert cols == expect_cols
    assert sp[-1] == 0                      # every benchmark tensor is a multiple of 8 elements
    assert tp[-1] >= 2 * 296 or cols == 512  # two tiles for every block, or the smallest tile


def test_invalid_tiling_arguments(B):
    for args in [([-1], 4), ([10], 0)]:
        with pytest.raises(B.AdaScaleError):
            B.tiling(*args)
    with pytest.raises(B.AdaScaleError):
        B.tiling([10], 4, grad_dtype=9)
