"""Parity of the CUDA library (through its C ABI) with the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)

import _harness as H  # noqa: E402
from paper_2007_05105_b200 import binding as B  # noqa: E402
from paper_2007_05105_b200 import synthetic  # noqa: E402

DEV = torch.device("cuda:0")
RAGGED = [1, 3, 4, 5, 7, 8, 9, 1023, 1025, 2048, 2049, 4097, 10000]


def _gen(seed):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    return g


# Bounds evidence: every gradient, parameter and momentum tensor of these tests sits between two
# guard zones of 256 poison bytes, and after each test the zones must be untouched.
GUARD_BYTES = 256
POISON = 0xA5
_guards = []


def _guarded(n, dtype, misalign=0):
    """n elements of `dtype` starting `misalign` elements past a 256-byte boundary, poison on both sides."""
    esz = torch.empty(0, dtype=dtype).element_size()
    g = GUARD_BYTES // esz
    whole = torch.empty(g + misalign + n + g, device=DEV, dtype=dtype)
    raw = whole.view(torch.uint8)
    raw[:(g + misalign) * esz] = POISON
    raw[(g + misalign + n) * esz:] = POISON
    _guards.append((raw, (g + misalign) * esz, (g + misalign + n) * esz))
    return whole[g + misalign:g + misalign + n]


@pytest.fixture(autouse=True)
def _guard_zones_stay_intact():
    _guards.clear()
    yield
    torch.cuda.synchronize()
    for raw, lo, hi in _guards:
        assert bool((raw[:lo] == POISON).all()) and bool((raw[hi:] == POISON).all()), "write outside a tensor"
    _guards.clear()


def _make_rows(numels, S, dtype, gen, k=3.0, mean_std=0.1, misalign=0):
    """Separate allocations per (row, tensor); `misalign` shifts every view by that many elements."""
    mean = [torch.empty(n, device=DEV).normal_(0, mean_std, generator=gen) for n in numels]
    rows = []
    for _ in range(S):
        row = []
        for n, m in zip(numels, mean):
            buf = torch.empty(n, device=DEV, dtype=torch.float32).normal_(0, 1, generator=gen)
            t = _guarded(n, dtype, misalign)
            t.copy_((m + k * mean_std * buf).to(dtype))
            row.append(t)
        rows.append(row)
    return rows


def _params(numels, gen, misalign=0):
    w, v = [], []
    for n in numels:
        w.append(_guarded(n, torch.float32, misalign).normal_(0, 1, generator=gen))
        v.append(_guarded(n, torch.float32, misalign).normal_(0, 0.1, generator=gen))
    return w, v


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("S", [1, 2, 3, 4, 5, 7, 8, 9, 16, 17, 32, 33, 40, 128])
def test_ragged_tensor_list(S, dtype):
    gen = _gen(1000 + S)
    name = "bf16" if dtype == torch.bfloat16 else "f32"
    pair = H.Pair(RAGGED, S, name, momentum=0.9, weight_decay=1e-3, lr={"kind": "const", "eta0": 0.05})
    w, v = _params(RAGGED, gen)
    pair.attach(w, v)
    for step in range(3):
        rows = _make_rows(RAGGED, S, dtype, gen, k=[0.5, 3.0, 10.0][step])
        pair.step(rows, "S=%d %s step %d" % (S, name, step))
    pair.close()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("runs", [1, 3, 8])
@pytest.mark.parametrize("S", [2, 8, 9, 16, 33])
def test_ragged_tensor_list_with_runs_from_the_counter(S, runs, dtype):
    """The tile hand-out of large jobs (runs of tiles from a device counter, sums added up by the
    producer warp), forced on a small ragged job plus one tensor of many tiles."""
    gen = _gen(2000 + 10 * S + runs)
    numels = RAGGED + [300000]
    name = "bf16" if dtype == torch.bfloat16 else "f32"
    pair = H.Pair(numels, S, name, momentum=0.9, weight_decay=1e-3, lr={"kind": "const", "eta0": 0.05}, tile_runs=runs)
    w, v = _params(numels, gen)
    pair.attach(w, v)
    for step in range(2):
        pair.step(_make_rows(numels, S, dtype, gen, k=[0.5, 10.0][step]), "S=%d runs=%d %s step %d" % (S, runs, name, step))
    pair.close()


def test_runs_from_the_counter_give_reproducible_sums_close_to_the_static_ones():
    gen = _gen(2100)
    numels = [200000, 4097, 77, 150016]
    rows = _make_rows(numels, 16, torch.float32, gen)
    w, v = _params(numels, gen)
    seen = {}
    for runs in (0, 1, 4, 4):
        ada = B.AdaScale(numels, 16, "f32", momentum=0.9)
        ada.set_tile_runs(runs)
        for _ in range(3):
            ada.reduce(rows, B.make_schedule())
        st = ada.get_gain_tau(True)
        seen.setdefault(runs, []).append((st.dev_sqsum, st.gbar_sqnorm, st.r))
        ada.close()
    assert seen[4][0] == seen[4][1]                       # bitwise, launch after launch and context after context
    for runs in (1, 4):                                     # other orders of the same terms: last bits only
        for a, b in zip(seen[runs][0], seen[0][0]):
            assert a == pytest.approx(b, rel=1e-13)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("misalign", [1, 2, 3])
def test_misaligned_pointers_take_the_scalar_path(misalign, dtype):
    gen = _gen(77 + misalign)
    numels = [5, 64, 1000, 4099]
    name = "bf16" if dtype == torch.bfloat16 else "f32"
    pair = H.Pair(numels, 5, name, momentum=0.5, weight_decay=0.01)
    w, v = _params(numels, gen, misalign)
    pair.attach(w, v)
    for step in range(2):
        pair.step(_make_rows(numels, 5, dtype, gen, misalign=misalign), "misalign %d step %d" % (misalign, step))
    pair.close()


def test_empty_tensors_are_skipped():
    gen = _gen(5)
    numels = [0, 17, 0, 256, 0]
    pair = H.Pair(numels, 4)
    w, v = _params(numels, gen)
    pair.attach(w, v)
    pair.step(_make_rows(numels, 4, torch.float32, gen), "empty")
    pair.close()


def test_identical_rows_zero_variance():
    gen = _gen(6)
    numels = [4096 + 5, 333]
    for S in (2, 3, 8, 32):
        base = [torch.empty(n, device=DEV).normal_(0, 1, generator=gen) for n in numels]
        rows = [[b.clone() for b in base] for _ in range(S)]
        pair = H.Pair(numels, S, theta=0.0)
        w, v = _params(numels, gen)
        pair.attach(w, v)
        st, ost = pair.step(rows, "identical S=%d" % S)
        assert st.dev_sqsum == 0.0 and st.sigma2_raw == 0.0
        assert abs(st.r - 1.0) < 1e-6
        pair.close()


def test_extreme_conditioning_k30_and_k0():
    """mu^2 is ~1/113 of ||gbar||^2 at k = 30, S = 8: the worst case for the subtraction."""
    gen = _gen(8)
    numels = [300000, 77]
    for k in (0.0, 0.3, 30.0, 300.0):
        pair = H.Pair(numels, 8, theta=0.0)
        w, v = _params(numels, gen)
        pair.attach(w, v)
        pair.step(_make_rows(numels, 8, torch.float32, gen, k=k), "k=%g" % k)
        pair.close()


def test_large_offset_small_noise():
    """Rows that agree to ~5 digits: the raw formula of App. B.3 would cancel, the shifted sums do not."""
    gen = _gen(9)
    n = 200000
    base = torch.empty(n, device=DEV).normal_(100.0, 1.0, generator=gen)
    rows = [[base + 1e-3 * torch.empty(n, device=DEV).normal_(0, 1, generator=gen)] for _ in range(8)]
    pair = H.Pair([n], 8, theta=0.0)
    w, v = _params([n], gen)
    pair.attach(w, v)
    pair.step(rows, "offset")
    pair.close()


def test_heavy_tailed_noise():
    wl = synthetic.workload("transformer_base")
    wl.shapes = [(50000,), (4096, 3), (17,)]
    src = synthetic.GradientSource(wl, device=DEV)
    wflat, vflat = src.init_params()
    pair = H.Pair(src.numels, wl.S, momentum=0.99, lr=wl.lr)
    pair.attach(src.views(wflat), src.views(vflat))
    for step in range(3):
        pair.step(src.fill(step), "student-t step %d" % step)
    pair.close()


@pytest.mark.parametrize("flags", [0, B.FLAG_LAGGED, B.FLAG_RATIO, B.FLAG_RATIO | B.FLAG_LAGGED, B.FLAG_CONT_TAU])
# the grid of App. C for S = 4: theta in {0, 1 - S/10, 1 - S/100, 1 - S/1000 (the rule, passed as -1), 1 - S/10000}
@pytest.mark.parametrize("theta", [0.0, 0.6, 0.96, -1.0, 0.9996])
def test_estimator_variants_and_theta(flags, theta):
    gen = _gen(11)
    numels = [5000, 129]
    lr = {"kind": "exp", "eta0": 0.08, "d": 0.0133, "T_S1": 50.0}
    pair = H.Pair(numels, 4, momentum=0.9, theta=theta, flags=flags, lr=lr)
    w, v = _params(numels, gen)
    pair.attach(w, v)
    for step in range(6):
        pair.step(_make_rows(numels, 4, torch.float32, gen, k=1.0 + step), "flags=%d step %d" % (flags, step),
                  compare_tensors=(step % 3 == 0))
    pair.close()


def test_step_schedule_crosses_its_boundaries():
    gen = _gen(12)
    numels = [3000]
    lr = {"kind": "step", "eta0": 0.1, "d": 0.1, "milestones": (5.0, 9.0, 14.0)}
    pair = H.Pair(numels, 8, momentum=0.9, theta=0.0, lr=lr)
    w, v = _params(numels, gen)
    pair.attach(w, v)
    seen = set()
    for step in range(8):
        st, _ = pair.step(_make_rows(numels, 8, torch.float32, gen, k=1.0), "sched step %d" % step)
        seen.add(round(st.lr, 12))
    assert len(seen) >= 3
    pair.close()


def test_elastic_scale_change():
    gen = _gen(13)
    numels = [2000, 31]
    pair = H.Pair(numels, 4, momentum=0.9, max_S=16)
    w, v = _params(numels, gen)
    pair.attach(w, v)
    for S in (4, 4, 8, 16, 16, 2):
        pair.dev.set_scale(S)
        pair.orc.set_scale(S)
        pair.step(_make_rows(numels, S, torch.float32, gen), "elastic S=%d" % S)
    with pytest.raises(B.AdaScaleError):
        pair.dev.set_scale(17)
    pair.close()


def test_nonfinite_gradients_skip_the_step():
    gen = _gen(14)
    numels = [1000, 10]
    pair = H.Pair(numels, 4, momentum=0.9)
    w, v = _params(numels, gen)
    pair.attach(w, v)
    pair.step(_make_rows(numels, 4, torch.float32, gen), "before")
    w0 = [t.clone() for t in w]
    v0 = [t.clone() for t in v]
    before = pair.dev.get_gain_tau(True)
    rows = _make_rows(numels, 4, torch.float32, gen)
    rows[2][0][17] = float("inf")
    pair.dev.step(rows, w, v, pair.sched_dev)
    st = pair.dev.get_gain_tau(True)
    assert st.status_bits & B.STATUS_NONFINITE and st.skipped == 1 and st.eta == 0.0
    assert st.tau == before.tau and st.t == before.t and st.sigma2_avg == before.sigma2_avg
    for a, b in zip(w + v, w0 + v0):
        assert torch.equal(a, b)
    # the oracle applies the same policy, and the next clean step is in step with it again
    rows_np = [[H.to_numpy_rows(g) for g in row] for row in rows]
    ost = pair.orc.step(rows_np, pair.w64, pair.v64, pair.sched_orc)
    assert ost["nonfinite"] == 1
    pair.step(_make_rows(numels, 4, torch.float32, gen), "after")
    assert pair.dev.get_gain_tau(True).status_bits == 0
    pair.close()


def test_bitwise_reproducible():
    gen = _gen(15)
    numels = [100000, 4097, 64]
    rows = _make_rows(numels, 8, torch.float32, gen)
    out = []
    for _ in range(2):
        g2 = _gen(16)
        w, v = _params(numels, g2)
        ada = B.AdaScale(numels, 8, momentum=0.9)
        sched = B.make_schedule("const", eta0=0.1)
        for _ in range(3):
            ada.step(rows, w, v, sched)
        st = ada.get_gain_tau(True)
        out.append((st.as_dict(), [t.clone() for t in w + v]))
        ada.close()
    assert out[0][0] == out[1][0]
    for a, b in zip(out[0][1], out[1][1]):
        assert torch.equal(a, b)


def test_checkpoint_resume_is_bitwise():
    gen = _gen(17)
    numels = [20000, 33]
    steps = [_make_rows(numels, 4, torch.float32, gen, k=1.0 + i) for i in range(6)]
    sched = B.make_schedule("exp", eta0=0.1, d=0.5, T_S1=10.0)

    def run(split):
        g2 = _gen(18)
        w, v = _params(numels, g2)
        ada = B.AdaScale(numels, 4, momentum=0.9, theta=0.6)
        for i, rows in enumerate(steps):
            if i == split:
                blob = ada.get_state()
                ada.close()
                ada = B.AdaScale(numels, 4, momentum=0.9, theta=0.6)
                ada.set_state(blob)
            ada.step(rows, w, v, sched)
        st = ada.get_gain_tau(True).as_dict()
        ada.close()
        return st, w, v

    a, b = run(None), run(3)
    assert a[0] == b[0]
    for x, y in zip(a[1] + a[2], b[1] + b[2]):
        assert torch.equal(x, y)
    with pytest.raises(B.AdaScaleError):
        ada = B.AdaScale(numels, 4)
        ada.set_state(b"\0" * B.STATE_BYTES)


def test_split_calls_equal_step_and_order_is_enforced():
    gen = _gen(19)
    numels = [5000]
    rows = _make_rows(numels, 4, torch.float32, gen)
    sched = B.make_schedule("const", eta0=0.1)
    res = []
    for split in (False, True):
        w, v = _params(numels, _gen(20))
        ada = B.AdaScale(numels, 4, momentum=0.9)
        if split:
            with pytest.raises(B.AdaScaleError) as e:
                ada.update(w, v)
            assert e.value.status == B.ERR_STATE
            ada.reduce(rows, sched)
            ada.update(w, v)
        else:
            ada.step(rows, w, v, sched)
        torch.cuda.synchronize()
        assert ada.launch_count == 2
        res.append((w[0].clone(), v[0].clone()))
        ada.close()
    assert torch.equal(res[0][0], res[1][0]) and torch.equal(res[0][1], res[1][1])


def test_host_gradients_entry_point():
    gen = _gen(21)
    numels = [3000, 64, 64, 100]
    rows = _make_rows(numels, 4, torch.float32, gen)
    sched = B.make_schedule("const", eta0=0.1)
    w1, v1 = _params(numels, _gen(22))
    w2, v2 = _params(numels, _gen(22))
    a = B.AdaScale(numels, 4, momentum=0.9)
    a.step(rows, w1, v1, sched)
    s1 = a.get_gain_tau(True)
    b = B.AdaScale(numels, 4, momentum=0.9)
    host = [[g.cpu().pin_memory() for g in row] for row in rows]
    s2 = b.step_host(host, w2, v2, sched)
    assert s1.as_dict() == s2.as_dict()
    for x, y in zip(w1 + v1, w2 + v2):
        assert torch.equal(x, y)
    a.close()
    b.close()


def test_error_paths_on_device():
    numels = [16]
    ada = B.AdaScale(numels, 2)
    sched = B.make_schedule()
    g = torch.zeros(64, device=DEV)
    w = torch.zeros(16, device=DEV)
    with pytest.raises(B.AdaScaleError) as e:
        ada.step([0, g.data_ptr()], [w], [w.clone()], sched)
    assert e.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.AdaScaleError) as e:
        ada.step([g.data_ptr() + 2, g.data_ptr()], [w], [w.clone()], sched)
    assert e.value.status == B.ERR_ALIGNMENT
    bad = B.make_schedule("exp", eta0=0.1, d=0.5, T_S1=0.0)
    with pytest.raises(B.AdaScaleError):
        ada.step([g, g], [w], [w.clone()], bad)
    ada.close()


def test_nonblocking_readback_trails_by_at_most_one_call():
    gen = _gen(23)
    numels = [1000]
    ada = B.AdaScale(numels, 2)
    w, v = _params(numels, gen)
    sched = B.make_schedule()
    rows = _make_rows(numels, 2, torch.float32, gen)
    assert ada.get_gain_tau(False).t == 0
    for _ in range(3):
        ada.step(rows, w, v, sched)
    ada.get_gain_tau(False)
    torch.cuda.synchronize()
    assert ada.get_gain_tau(False).t == 3
    ada.close()


# ---------------------------------------------------------------- one-pass (fused, lagged) mode

FUSED = B.FLAG_LAGGED | B.FLAG_FUSED


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("S", [1, 2, 3, 5, 8, 16, 17, 32, 40])
def test_fused_mode_against_the_lagged_oracle(S, dtype):
    gen = _gen(3000 + S)
    name = "bf16" if dtype == torch.bfloat16 else "f32"
    lr = {"kind": "exp", "eta0": 0.05, "d": 0.5, "T_S1": 20.0}
    pair = H.Pair(RAGGED, S, name, momentum=0.9, weight_decay=1e-3, flags=FUSED, lr=lr)
    w, v = _params(RAGGED, gen)
    pair.attach(w, v)
    for step in range(4):
        rows = _make_rows(RAGGED, S, dtype, gen, k=[0.5, 3.0, 10.0, 1.0][step])
        st, _ = pair.step(rows, "fused S=%d %s step %d" % (S, name, step))
    if S > 1:
        assert st.r > 1.0  # the gain follows the averages from the second step on
    pair.close()


@pytest.mark.parametrize("runs", [1, 4])
@pytest.mark.parametrize("S", [3, 16, 40])
def test_fused_mode_with_runs_from_the_counter(S, runs):
    gen = _gen(4150 + S + runs)
    numels = RAGGED + [250000]
    pair = H.Pair(numels, S, "bf16", momentum=0.9, weight_decay=1e-3, flags=FUSED, lr={"kind": "const", "eta0": 0.05},
                  tile_runs=runs)
    w, v = _params(numels, gen)
    pair.attach(w, v)
    for step in range(3):
        pair.step(_make_rows(numels, S, torch.bfloat16, gen, k=1.0 + step), "fused S=%d runs=%d step %d" % (S, runs, step))
    pair.close()


@pytest.mark.parametrize("misalign", [1, 3])
def test_fused_mode_with_misaligned_gradients_and_parameters(misalign):
    gen = _gen(3100 + misalign)
    numels = [5, 64, 1000, 4099]
    for grads_off, params_off in [(misalign, 0), (0, misalign), (misalign, misalign)]:
        pair = H.Pair(numels, 4, "f32", momentum=0.5, weight_decay=0.01, flags=FUSED)
        w, v = _params(numels, gen, params_off)
        pair.attach(w, v)
        for step in range(2):
            pair.step(_make_rows(numels, 4, torch.float32, gen, misalign=grads_off), "fused misalign step %d" % step)
        pair.close()


def test_fused_mode_is_bitwise_the_two_kernel_lagged_mode():
    gen = _gen(3200)
    numels = [100000, 4097, 64, 7]
    steps = [_make_rows(numels, 8, torch.bfloat16, gen, k=1.0 + i) for i in range(4)]
    sched = B.make_schedule("step", eta0=0.1, d=0.1, milestones=(3.0,))
    out = []
    for flags in (B.FLAG_LAGGED, FUSED):
        w, v = _params(numels, _gen(3201))
        ada = B.AdaScale(numels, 8, "bf16", momentum=0.9, weight_decay=1e-4, flags=flags)
        for rows in steps:
            ada.step(rows, w, v, sched)
        out.append((ada.get_gain_tau(True).as_dict(), w, v, ada.launch_count))
        ada.close()
    assert out[0][0] == out[1][0]
    for a, b in zip(out[0][1] + out[0][2], out[1][1] + out[1][2]):
        assert torch.equal(a, b)
    assert out[0][3] == 8 and out[1][3] == 4      # two launches per step against one


def test_fused_mode_call_rules():
    with pytest.raises(B.AdaScaleError) as e:
        B.AdaScale([16], 2, flags=B.FLAG_FUSED)   # needs the lagged estimate
    assert e.value.status == B.ERR_INVALID_ARG
    ada = B.AdaScale([16], 2, flags=FUSED)
    g = torch.zeros(16, device=DEV)
    w = torch.zeros(16, device=DEV)
    v = torch.zeros(16, device=DEV)
    sched = B.make_schedule()
    ada.step([g, g], [w], [v], sched)
    for call in (lambda: ada.reduce([g, g], sched), lambda: ada.update([w], [v]), lambda: ada.mean_grad()):
        with pytest.raises(B.AdaScaleError) as e:
            call()
        assert e.value.status == B.ERR_STATE
    ada.close()


def test_one_tensor_with_more_than_2_31_elements():
    """64-bit offsets: a single bf16 tensor of 2^31 + 4101 elements, S = 2, rows x and -x.

    Too large for the CPU oracle in test time; the expected values follow from the construction:
    gbar = 0 exactly, so N = 0, D = 2 sum x^2 (torch fp64 reduction, an independent routine),
    v <- rho v + lambda w and w <- w - eta v.
    """
    n = (1 << 31) + 4101
    gen = _gen(4000)
    x = torch.empty(n, device=DEV, dtype=torch.bfloat16)
    for lo in range(0, n, 1 << 28):
        hi = min(n, lo + (1 << 28))
        x[lo:hi] = torch.empty(hi - lo, device=DEV).normal_(0, 1, generator=gen).to(torch.bfloat16)
    neg = -x
    w = torch.full((n,), 2.0, device=DEV)
    v = torch.full((n,), 0.5, device=DEV)
    ada = B.AdaScale([n], 2, "bf16", momentum=0.5, weight_decay=0.25, theta=0.0)
    ada.step([[x], [neg]], [w], [v], B.make_schedule("const", eta0=0.125))
    st = ada.get_gain_tau(True)
    sq = 0.0
    for lo in range(0, n, 1 << 28):
        sq += float(x[lo:min(n, lo + (1 << 28))].double().pow(2).sum())
    assert st.gbar_sqnorm == 0.0
    assert st.dev_sqsum == pytest.approx(2.0 * sq, rel=1e-6)
    # sigma^2 = D, mu^2 = -D/2 -> clamped to 0 -> r = S = 2, eta = 0.25; v = 0.25 + 0.5 = 0.75, w = 2 - 0.1875
    assert st.r == pytest.approx(2.0, rel=1e-12) and st.eta == pytest.approx(0.25, rel=1e-12)
    gbar = ada.mean_grad_tensors()[0]
    for sl in (slice(0, 4096), slice((1 << 31) - 2048, (1 << 31) + 2048), slice(n - 4101, n)):
        assert bool((gbar[sl] == 0).all())
        assert bool((v[sl] == 0.75).all()) and bool((w[sl] == 2.0 - 0.25 * 0.75).all())
    assert float(v.min()) == 0.75 and float(v.max()) == 0.75
    assert float(w.min()) == 1.8125 and float(w.max()) == 1.8125
    ada.close()


def test_scale_of_one_thousand_rows():
    """S = 1000: many row chunks per tile, and the paper's theta rule gives 0 (no averaging)."""
    gen = _gen(4100)
    numels = [3000, 7]
    # r is several hundred here, so the base rate is small: eta_t = r_t * lr stays of order 0.01-0.1
    pair = H.Pair(numels, 1000, "f32", momentum=0.9, lr={"kind": "const", "eta0": 1e-4})
    assert pair.orc.theta == 0.0
    w, v = _params(numels, gen)
    pair.attach(w, v)
    for step in range(2):
        st, _ = pair.step(_make_rows(numels, 1000, torch.float32, gen, k=30.0), "S=1000 step %d" % step)
    assert 1.0 <= st.r <= 1000.0
    pair.close()


def test_steps_replayed_from_a_cuda_graph_match_eager_steps():
    """adascale_step only enqueues, so once its tables are on the device it can be captured."""
    gen = _gen(4200)
    numels = [50000, 4097, 64]
    rows = _make_rows(numels, 8, torch.float32, gen)
    other = _make_rows(numels, 8, torch.float32, gen)
    sched = B.make_schedule("exp", eta0=0.05, d=0.5, T_S1=20.0)

    def fresh():
        w, v = _params(numels, _gen(4201))
        return B.AdaScale(numels, 8, momentum=0.9, weight_decay=1e-4), w, v

    eager, we, ve = fresh()
    for _ in range(4):
        eager.step(rows, we, ve, sched)
    ref = eager.get_gain_tau(True).as_dict()

    ada, w, v = fresh()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        ada.step(rows, w, v, sched, stream=side.cuda_stream)       # step 1, eager: uploads tables and tiling
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            ada.step(rows, w, v, sched, stream=side.cuda_stream)   # captured once ...
            with pytest.raises(B.AdaScaleError) as e:              # ... new pointers are refused, nothing enqueued
                ada.step(other, w, v, sched, stream=side.cuda_stream)
            assert e.value.status == B.ERR_STATE
        for _ in range(3):                                          # ... replayed as steps 2, 3, 4
            graph.replay()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    got = ada.get_gain_tau(True).as_dict()
    assert got == ref
    for a, b in zip(w + v, we + ve):
        assert torch.equal(a, b)
    eager.close()
    ada.close()


def test_fused_mode_with_elastic_scale_host_gradients_and_resume():
    gen = _gen(4300)
    numels = [6000, 31]
    lr = {"kind": "step", "eta0": 0.05, "d": 0.5, "milestones": (6.0,)}
    pair = H.Pair(numels, 4, "bf16", momentum=0.9, weight_decay=1e-3, flags=FUSED, max_S=16, lr=lr)
    w, v = _params(numels, gen)
    pair.attach(w, v)
    for S in (4, 8, 16, 2):
        pair.dev.set_scale(S)
        pair.orc.set_scale(S)
        pair.step(_make_rows(numels, S, torch.bfloat16, gen), "fused elastic S=%d" % S)
    # resume in a new context, and feed the next step from host memory
    blob = pair.dev.get_state()
    ada = B.AdaScale(numels, 2, "bf16", momentum=0.9, weight_decay=1e-3, flags=FUSED, max_S=16)
    ada.set_state(blob)
    rows = _make_rows(numels, 2, torch.bfloat16, gen)
    w2, v2 = [t.clone() for t in w], [t.clone() for t in v]
    pair.dev.step(rows, w, v, pair.sched_dev)
    a = pair.dev.get_gain_tau(True).as_dict()
    b = ada.step_host([[g.cpu().pin_memory() for g in row] for row in rows], w2, v2, pair.sched_dev).as_dict()
    assert a == b
    for x, y in zip(w + v, w2 + v2):
        assert torch.equal(x, y)
    ada.close()
    pair.close()


@pytest.mark.parametrize("runs", [-1, 2])
def test_two_column_shards_reproduce_the_unsharded_step(runs):
    """Column-sharded use emulated on one GPU: two contexts over the two halves of the tensor
    list, their sums added on the device (what an all-reduce of 16 bytes would do), then the
    scalar part and the update per shard.  No kernel waits for another: the calls are sequential.
    With runs forced, the shards' reduce kernels keep a last block that adds up the run pairs."""
    gen = _gen(4400)
    numels = [30000, 4097, 64, 7, 2048, 12345]
    split = 3
    steps = [_make_rows(numels, 8, torch.float32, gen, k=1.0 + i) for i in range(3)]
    lr = {"kind": "exp", "eta0": 0.05, "d": 0.5, "T_S1": 10.0}
    sched = H.device_lr(lr)

    pair = H.Pair(numels, 8, "f32", momentum=0.9, weight_decay=1e-3, lr=lr)      # unsharded device + oracle
    w, v = _params(numels, _gen(4401))
    pair.attach(w, v)

    ws, vs = _params(numels, _gen(4401))
    shards = [B.AdaScale(numels[:split], 8, momentum=0.9, weight_decay=1e-3),
              B.AdaScale(numels[split:], 8, momentum=0.9, weight_decay=1e-3)]
    for ada in shards:
        ada.set_tile_runs(runs)
    parts = [slice(0, split), slice(split, len(numels))]
    sums = [torch.zeros(2, dtype=torch.float64, device=DEV) for _ in shards]
    for i, rows in enumerate(steps):
        pair._push_state = lambda tensors=None: None      # free-running here: compare the two device paths
        st, ost = pair.step(rows, "unsharded step %d" % i, compare_tensors=False)
        for ada, part, buf in zip(shards, parts, sums):
            ada.reduce_sums([row[part] for row in rows], buf)
        total = sums[0] + sums[1]                          # the exchange
        for ada, part in zip(shards, parts):
            ada.apply_sums(total, sched, ws[part], vs[part])
        a, b = shards[0].get_gain_tau(True), shards[1].get_gain_tau(True)
        assert a.as_dict() == b.as_dict()                  # every shard sees the identical scalars
        for name in ("r", "tau", "eta", "sigma2_raw", "mu2_raw", "gbar_sqnorm", "dev_sqsum"):
            assert getattr(a, name) == pytest.approx(getattr(st, name), rel=1e-12), name
            assert getattr(a, name) == pytest.approx(ost[name] if name in ost else getattr(st, name), rel=1e-5)
    for x, y in zip(w + v, ws + vs):
        torch.testing.assert_close(x, y, rtol=1e-6, atol=1e-9)
    for ada in shards:
        ada.close()
    pair.close()
