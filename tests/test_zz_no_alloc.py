"""The entry point that allocates nothing, checked against the context-based one.

Some users of this library cannot allocate device memory when they need the gradient
statistics (all of it already belongs to another allocator, or allocation after start-up is
ruled out because it can fail late or stall the device).  ``adascale_grad_stats_static``
serves them: inputs and outputs are the caller's buffers and the library's scratch is a fixed
array inside the library.  This test calls it through the C ABI twice in a row, with different
sizes, row counts and element types, and compares the mean gradient and the two sums with what
``adascale_reduce`` produces for the same rows, within the tolerances of the parity tests; a
second test compares it with the CPU oracle over the corner sizes (one row, two rows, the
largest row count, fewer elements than one vector) with poisoned guard zones around the
caller's output buffers.  The file is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)

import oracle  # noqa: E402
import _harness as H  # noqa: E402
from paper_2007_05105_b200 import binding as B  # noqa: E402

DEV = torch.device("cuda:0")


def _reference(rows, n, name):
    """The same statistics through the context API (which allocates)."""
    ada = B.AdaScale([n], len(rows), name)
    ada.reduce([[r] for r in rows], B.make_schedule())
    st = ada.get_gain_tau(True)
    gbar = ada.mean_grad_tensors()[0].clone()
    ada.close()
    return gbar, st.dev_sqsum, st.gbar_sqnorm


def _check(rows, n, name):
    # the caller's own buffers: nothing is allocated inside the call
    gbar = torch.full((n + 8,), float("nan"), device=DEV)[:n]
    sums = torch.full((2,), float("nan"), dtype=torch.float64, device=DEV)
    B.grad_stats_static(rows, n, name, gbar, sums)
    torch.cuda.synchronize()
    ref_gbar, ref_D, ref_N = _reference(rows, n, name)
    D, N = sums.tolist()
    Q = ref_D + len(rows) * ref_N                     # sum_i ||g_i||^2
    assert abs(D - ref_D) <= 1e-5 * abs(ref_D) + 1e-12 * Q
    assert abs(N - ref_N) <= 1e-5 * abs(ref_N) + 1e-12 * Q
    scale = torch.stack([r.float().abs() for r in rows]).max(dim=0).values
    err = (gbar - ref_gbar).abs()
    assert bool((err <= 3e-7 * scale + 1e-45).all()), float((err / (3e-7 * scale + 1e-45)).max())


def test_static_entry_point_matches_the_context_api_twice_in_a_row():
    gen = torch.Generator(device=DEV)
    gen.manual_seed(2007)
    for S, n, dtype, name in [(8, 300007, torch.float32, "f32"), (5, 70001, torch.bfloat16, "bf16")]:
        mean = torch.empty(n, device=DEV).normal_(0, 0.1, generator=gen)
        rows = [(mean + 0.3 * torch.empty(n, device=DEV).normal_(0, 1, generator=gen)).to(dtype) for _ in range(S)]
        _check(rows, n, name)


GUARD = 256  # bytes of poison either side of an output buffer


def _guarded(nbytes):
    """A device byte buffer with 0xA5-filled guard zones; returns (whole, payload view)."""
    whole = torch.full((nbytes + 2 * GUARD,), 0xA5, dtype=torch.uint8, device=DEV)
    return whole, whole[GUARD:GUARD + nbytes]


def _guards_intact(whole, nbytes):
    return bool((whole[:GUARD] == 0xA5).all()) and bool((whole[GUARD + nbytes:] == 0xA5).all())


@pytest.mark.parametrize("name", ["f32", "bf16"])
@pytest.mark.parametrize("S", [1, 2, 3, 32])
def test_static_entry_point_matches_the_oracle_at_the_corner_sizes(S, name):
    gen = torch.Generator(device=DEV)
    gen.manual_seed(500 + S)
    dtype = torch.bfloat16 if name == "bf16" else torch.float32
    for n in (1, 7, 8, 300007):
        mean = torch.empty(n, device=DEV).normal_(0, 0.1, generator=gen)
        rows = [(mean + 0.3 * torch.empty(n, device=DEV).normal_(0, 1, generator=gen)).to(dtype) for _ in range(S)]
        gw, gpay = _guarded(4 * n)
        sw, spay = _guarded(16)
        B.grad_stats_static(rows, n, name, gpay.data_ptr(), spay.data_ptr())
        torch.cuda.synchronize()
        assert _guards_intact(gw, 4 * n) and _guards_intact(sw, 16), "write outside the caller's buffers"
        gbar = gpay.view(torch.float32).cpu().numpy()
        D, N = spay.view(torch.float64).tolist()
        rows_np = [H.to_numpy_rows(r) for r in rows]
        ogbar, oD, oN, oQ = oracle.grad_stats(rows_np, True, H.NTHREADS)
        label = "S=%d n=%d %s" % (S, n, name)
        assert abs(D - oD) <= 1e-5 * abs(oD) + 1e-12 * oQ, (label, D, oD)
        assert abs(N - oN) <= 1e-5 * abs(oN) + 1e-12 * oQ, (label, N, oN)
        H.check_gbar(gbar, ogbar, H.row_scale(rows_np), label, H.gbar_ulps(S))


def test_static_entry_point_rejects_what_it_cannot_hold():
    g = torch.zeros(64, device=DEV)
    sums = torch.zeros(2, dtype=torch.float64, device=DEV)
    with pytest.raises(B.AdaScaleError) as e:
        B.grad_stats_static([g] * (B.STATIC_MAX_ROWS + 1), 64, "f32", g, sums)
    assert e.value.status == B.ERR_TOO_LARGE and "maximum" in str(e.value)
    with pytest.raises(B.AdaScaleError) as e:
        B.grad_stats_static([g, g], B.STATIC_MAX_NUMEL + 1, "f32", g, sums)
    assert e.value.status == B.ERR_TOO_LARGE
    with pytest.raises(B.AdaScaleError) as e:
        B.grad_stats_static([g, g.data_ptr() + 4], 32, "f32", g, sums)
    assert e.value.status == B.ERR_ALIGNMENT
    with pytest.raises(B.AdaScaleError) as e:
        B.grad_stats_static([g, g], 0, "f32", g, sums)
    assert e.value.status == B.ERR_INVALID_ARG
