"""The synthetic workloads have the tensor lists and sizes the benchmark configurations name."""
import numpy as np
import pytest
import torch

from paper_2007_05105_b200 import synthetic


@pytest.mark.parametrize("name,P,T,S,dtype", [
    ("single_1m", 1048576, 1, 4, "f32"),
    ("resnet18", 11689512, 62, 8, "f32"),
    ("resnet50", 25557032, 161, 16, "bf16"),
    ("transformer_base", 60917760, 257, 32, "f32"),
    ("decoder_24l", 354823168, 292, 32, "bf16"),
])
def test_parameter_counts(name, P, T, S, dtype):
    wl = synthetic.workload(name)
    assert (wl.P, len(wl.shapes), wl.S, wl.grad_dtype) == (P, T, S, dtype)


def test_drift_schedule_is_linear():
    wl = synthetic.workload("decoder_24l")
    assert wl.k_at(0) == pytest.approx(0.1) and wl.k_at(199) == pytest.approx(10.0)
    assert wl.k_at(100) == pytest.approx(0.1 + 9.9 * 100 / 199)


def test_source_is_seeded_and_has_the_stated_moments():
    wl = synthetic.workload("resnet18")
    wl.shapes = synthetic.resnet18_shapes(width=16, classes=10)
    a = synthetic.GradientSource(wl)
    b = synthetic.GradientSource(wl)
    ga, gb = a.fill(3), b.fill(3)
    for ra, rb in zip(ga, gb):
        for x, y in zip(ra, rb):
            assert torch.equal(x, y)
    g0 = torch.cat([t.reshape(-1) for t in ga[0]])
    g1 = torch.cat([t.reshape(-1) for t in ga[1]])
    m = torch.cat([t.reshape(-1) for t in a.views(a.mean)])
    assert float(m.std()) == pytest.approx(0.1, rel=0.02)
    assert float((g0 - m).std()) == pytest.approx(0.3, rel=0.02)     # s = k * std(m), k = 3
    assert abs(float(np.corrcoef((g0 - m).numpy(), (g1 - m).numpy())[0, 1])) < 0.01


def test_student_noise_has_unit_variance_and_heavy_tails():
    wl = synthetic.workload("transformer_base")
    wl.shapes = [(400000,)]
    src = synthetic.GradientSource(wl)
    g = src.fill(0)[0][0]
    n = (g - src.views(src.mean)[0]) / (3.0 * 0.1)
    assert float(n.median().abs()) < 0.01
    # Student-t(3)/sqrt(3): P(|x| > 4) is about 1.3e-3... far above the normal's 6e-5
    assert float((n.abs() > 4).float().mean()) > 5e-4
    core = n[n.abs() < 20]
    assert float(core.var()) == pytest.approx(1.0, rel=0.25)


def test_bf16_rows_are_rounded_values():
    wl = synthetic.workload("resnet50")
    wl.shapes = [(1000,)]
    src = synthetic.GradientSource(wl)
    g = src.fill(0)[0][0]
    assert g.dtype == torch.bfloat16
