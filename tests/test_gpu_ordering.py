"""Ordering of overlapped launches, the give-up path of the bounded waits, and guard zones.

The step's kernels overlap through programmatic dependent launch.  These tests run many steps
back to back with nothing else on the stream (the situation in which a kernel can start while
its predecessors drain) and require the parameters and the momentum to be bitwise those of the
same steps run with a stream synchronisation after every launch, and within tolerance of the
oracle's fp64 trajectory.  A stale read would lose an update for a tile, which is hundreds of
times the tolerance.
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
from paper_2007_05105_b200 import synthetic  # noqa: E402

DEV = torch.device("cuda:0")
FUSED = B.FLAG_LAGGED | B.FLAG_FUSED


def _run(wl, src, grads, w0, v0, steps, flags, sync_every_launch, tile_runs=-1):
    """`steps` iterations on fixed gradient buffers; returns (w, v, stats) as host arrays."""
    w, v = w0.clone(), v0.clone()
    wv, vv = src.views(w), src.views(v)
    ada = B.AdaScale(src.numels, wl.S, wl.grad_dtype, momentum=wl.momentum, weight_decay=wl.weight_decay, flags=flags)
    ada.set_tile_runs(tile_runs)
    sched = H.device_lr(wl.lr)
    gp, wp, vp = B.pointer_array(grads), B.pointer_array(wv), B.pointer_array(vv)
    stream = torch.cuda.current_stream(DEV).cuda_stream
    torch.cuda.synchronize()
    for _ in range(steps):
        if sync_every_launch and not (flags & B.FLAG_FUSED):
            ada.reduce(gp, sched, stream)
            torch.cuda.synchronize()
            ada.update(wp, vp, stream)
            torch.cuda.synchronize()
        else:
            ada.step(gp, wp, vp, sched, stream)
            if sync_every_launch:
                torch.cuda.synchronize()
    st = ada.get_gain_tau(True)
    out = (w.cpu().numpy(), v.cpu().numpy(), st)
    ada.close()
    return out


def _oracle_run(wl, src, grads, w0, v0, steps, lagged):
    orc = oracle.Oracle(wl.S, momentum=wl.momentum, weight_decay=wl.weight_decay, nthreads=H.NTHREADS,
                        flags=oracle.FLAG_LAGGED if lagged else 0)
    rows = [[H.to_numpy_rows(g) for g in row] for row in grads]
    w64 = [t.cpu().numpy().astype(np.float64) for t in src.views(w0)]
    v64 = [t.cpu().numpy().astype(np.float64) for t in src.views(v0)]
    lr = H.oracle_lr(wl.lr)
    orc.reduce(rows)          # fixed gradients: the sums are those of every iteration
    for _ in range(steps):
        st = orc.scalar(lr)
        orc.update(w64, v64)
    return w64, v64, st


@pytest.mark.parametrize("name,steps", [("single_1m", 400), ("resnet18", 300)])
@pytest.mark.parametrize("flags", [0, B.FLAG_GRADS_READY, FUSED, FUSED | B.FLAG_GRADS_READY],
                         ids=["default", "grads_ready", "fused", "fused_grads_ready"])
def test_back_to_back_steps_equal_synchronised_steps(name, steps, flags):
    wl = synthetic.workload(name)
    wl.lr = {"kind": "const", "eta0": 0.01}   # a constant learning rate keeps every step's update the same size
    src = synthetic.GradientSource(wl, device=DEV)
    grads = src.fill(0)
    w0, v0 = src.init_params()
    w_a, v_a, st_a = _run(wl, src, grads, w0, v0, steps, flags, sync_every_launch=False)
    w_b, v_b, st_b = _run(wl, src, grads, w0, v0, steps, flags, sync_every_launch=True)
    assert st_a.t == steps and st_a.status_bits == 0
    assert st_a.tau == st_b.tau and st_a.r == st_b.r
    assert np.array_equal(w_a.view(np.uint32), w_b.view(np.uint32)), "w differs between overlapped and synchronised steps"
    assert np.array_equal(v_a.view(np.uint32), v_b.view(np.uint32)), "v differs between overlapped and synchronised steps"
    # and the synchronised run is the right trajectory: fp64 oracle, same fixed gradients
    w64, v64, ost = _oracle_run(wl, src, grads, w0, v0, steps, lagged=bool(flags & B.FLAG_LAGGED))
    assert abs(st_a.tau - ost["tau"]) <= 1e-5 * ost["tau"]
    # Free-running fp32 storage against fp64: 1e-5 of the values and of the distance travelled, plus
    # the mean gradient's own fp32 summation error (a few ulps of max_i |g_ij|), which the momentum
    # sums to 1/(1 - rho) times itself and every step carries into w.  One lost update of a tile
    # would be eta |v|, hundreds of times this.
    w0_views = [t.cpu().numpy().astype(np.float64) for t in src.views(w0)]
    rows = [[H.to_numpy_rows(g) for g in row] for row in grads]
    eta = ost["eta"]
    for k, (o, n) in enumerate(zip(src.offsets, src.numels)):
        gerr = 20 * 2.0 ** -24 * H.row_scale([row[k] for row in rows]) / (1.0 - wl.momentum)
        moved = np.abs(w64[k] - w0_views[k])
        tol = 1e-5 * (np.abs(w64[k]) + moved) + steps * eta * gerr + 1e-12
        err = np.abs(w_a[o:o + n].astype(np.float64) - w64[k])
        assert (err <= tol).all(), "tensor %d: worst %g x tolerance" % (k, float((err / tol).max()))
        assert (err > 0.1 * eta * np.abs(v64[k])).mean() < 0.05, "tolerance would hide a lost update"
        tol_v = 1e-5 * np.abs(v64[k]) + gerr + 1e-12
        err_v = np.abs(v_a[o:o + n].astype(np.float64) - v64[k])
        assert (err_v <= tol_v).all(), "tensor %d momentum: worst %g x tolerance" % (k, float((err_v / tol_v).max()))


@pytest.mark.parametrize("flags", [0, B.FLAG_GRADS_READY, FUSED, FUSED | B.FLAG_GRADS_READY],
                         ids=["default", "grads_ready", "fused", "fused_grads_ready"])
@pytest.mark.parametrize("runs", [1, 4])
def test_back_to_back_steps_with_runs_from_the_counter(runs, flags):
    """The same requirement with the tile hand-out of large jobs forced on resnet18: the run counter is
    shared by consecutive launches, so a launch that touched it too early would process tiles twice."""
    wl = synthetic.workload("resnet18")
    wl.lr = {"kind": "const", "eta0": 0.01}
    src = synthetic.GradientSource(wl, device=DEV)
    grads = src.fill(0)
    w0, v0 = src.init_params()
    w_a, v_a, st_a = _run(wl, src, grads, w0, v0, 200, flags, False, runs)
    w_b, v_b, st_b = _run(wl, src, grads, w0, v0, 200, flags, True, runs)
    assert st_a.t == 200 and st_a.status_bits == 0 and st_a.tau == st_b.tau
    assert np.array_equal(w_a.view(np.uint32), w_b.view(np.uint32))
    assert np.array_equal(v_a.view(np.uint32), v_b.view(np.uint32))
    w_c, v_c, st_c = _run(wl, src, grads, w0, v0, 200, flags, True, 0)        # static assignment
    assert st_a.tau == pytest.approx(st_c.tau, rel=1e-12)
    np.testing.assert_allclose(w_a, w_c, rtol=1e-5, atol=1e-7)


def test_update_tiles_one_per_block_back_to_back():
    """A job with fewer update tiles than blocks: every block's only tile is its prefetched first tile."""
    wl = synthetic.workload("single_1m")
    wl.shapes = [(300 * 1024,)]
    wl.lr = {"kind": "const", "eta0": 0.02}
    src = synthetic.GradientSource(wl, device=DEV)
    grads = src.fill(0)
    w0, v0 = src.init_params()
    w_a, v_a, _ = _run(wl, src, grads, w0, v0, 500, 0, False)
    w_b, v_b, _ = _run(wl, src, grads, w0, v0, 500, 0, True)
    assert np.array_equal(w_a.view(np.uint32), w_b.view(np.uint32))
    assert np.array_equal(v_a.view(np.uint32), v_b.view(np.uint32))


# ------------------------------------------------------------------ bounded waits


def _small_job(flags=0):
    numels = [70000, 33, 4096, 150001]
    gen = torch.Generator(device=DEV)
    gen.manual_seed(99)
    S = 8
    mean = [torch.empty(n, device=DEV).normal_(0, 0.1, generator=gen) for n in numels]
    rows = [[m + 0.3 * torch.empty_like(m).normal_(0, 1, generator=gen) for m in mean] for _ in range(S)]
    w = [torch.empty(n, device=DEV).normal_(0, 1, generator=gen) for n in numels]
    v = [torch.empty(n, device=DEV).normal_(0, 0.1, generator=gen) for n in numels]
    return numels, S, rows, w, v


@pytest.mark.parametrize("runs", [-1, 2])
@pytest.mark.parametrize("polls", [0, 1])
def test_a_wait_that_runs_out_is_reported_and_changes_nothing(polls, runs):
    """The handshake waits of the reduce kernel are given a limit that cannot (0 polls) or can hardly
    (1 poll) be met.  The step must return, report the condition, leave w and v alone, and keep
    skipping; a fresh context on the same device then passes a parity step."""
    numels, S, rows, w, v = _small_job()
    w_before = [t.clone() for t in w]
    v_before = [t.clone() for t in v]
    ada = B.AdaScale(numels, S, "f32", momentum=0.9, weight_decay=1e-3)
    sched = B.make_schedule("const", eta0=0.1)
    ada.set_tile_runs(runs)
    ada.set_wait_limit(polls)
    ada.step(rows, w, v, sched)
    st = ada.get_gain_tau(True)
    torch.cuda.synchronize()
    if polls == 0:
        assert st.status_bits & B.STATUS_WAIT_TIMEOUT
    if st.status_bits & B.STATUS_WAIT_TIMEOUT:
        assert st.t == 0 and st.tau == 0.0 and st.skipped == 1 and st.eta == 0.0
        for a, b in zip(w + v, w_before + v_before):
            assert torch.equal(a, b)
        # the condition is sticky: later steps are skipped too, even with the default limit
        ada.set_wait_limit(1 << 22)
        ada.step(rows, w, v, sched)
        st2 = ada.get_gain_tau(True)
        assert st2.status_bits & B.STATUS_WAIT_TIMEOUT and st2.t == 0 and st2.skipped == 2
        for a, b in zip(w + v, w_before + v_before):
            assert torch.equal(a, b)
    else:  # one poll happened to be enough everywhere: then the step is an ordinary, valid one
        assert st.t == 1 and st.r >= 1.0
    ada.close()
    # the device and a fresh context are fine afterwards
    pair = H.Pair(numels, S, "f32", momentum=0.9, weight_decay=1e-3)
    pair.attach(w, v)
    pair.step(rows, "after a timed-out context")
    pair.close()


def test_wait_timeout_in_the_one_pass_mode_is_reported():
    numels, S, rows, w, v = _small_job()
    ada = B.AdaScale(numels, S, "f32", momentum=0.9, flags=FUSED)
    ada.set_wait_limit(0)
    ada.step(rows, w, v, B.make_schedule("const", eta0=0.1))
    st = ada.get_gain_tau(True)
    assert st.status_bits & B.STATUS_WAIT_TIMEOUT and st.t == 0 and st.skipped == 1
    ada.close()


def test_set_state_clears_a_timeout():
    numels, S, rows, w, v = _small_job()
    ada = B.AdaScale(numels, S, "f32", momentum=0.9)
    sched = B.make_schedule("const", eta0=0.1)
    ada.step(rows, w, v, sched)
    blob = ada.get_state()
    ada.set_wait_limit(0)
    ada.step(rows, w, v, sched)
    assert ada.get_gain_tau(True).status_bits & B.STATUS_WAIT_TIMEOUT
    ada.set_wait_limit(1 << 22)
    ada.set_state(blob)
    ada.step(rows, w, v, sched)
    st = ada.get_gain_tau(True)
    assert st.status_bits == 0 and st.t == 2
    ada.close()


# ---- the scalar part left open by a reduce launch -------------------------------------------

def _open_job(seed, S=8, k=1.0):
    gen = torch.Generator(device=DEV)
    gen.manual_seed(seed)
    numels = [30000, 4097, 64, 5]
    m = [0.1 * torch.randn(n, device=DEV, generator=gen) for n in numels]
    rows = [[m[j] + k * 0.1 * torch.randn(n, device=DEV, generator=gen) for j, n in enumerate(numels)] for _ in range(S)]
    w = [torch.randn(n, device=DEV, generator=gen) for n in numels]
    v = [torch.zeros(n, device=DEV) for n in numels]
    return numels, rows, w, v


def test_a_reduce_call_without_an_update_still_completes_its_iteration():
    """On small jobs the reduce kernel stops at one pair of sums per block and the next kernel does
    the scalar part: the update kernel when one follows, a one-block kernel when the caller asks
    for the statistics (or reduces again) first.  Whichever completes it, the state is the same."""
    numels, rows, w0, v0 = _open_job(77)
    _, rows2, _, _ = _open_job(78, k=3.0)
    sched = B.make_schedule("step", eta0=0.1, d=0.5, milestones=(1.0, 3.0))
    kw = dict(momentum=0.9, weight_decay=1e-4)

    ref = B.AdaScale(numels, 8, **kw)
    w, v = [t.clone() for t in w0], [t.clone() for t in v0]
    ref.step(rows, w, v, sched)
    one = ref.get_gain_tau(True).as_dict()
    w_one, v_one = [t.clone() for t in w], [t.clone() for t in v]
    ref.step(rows2, w, v, sched)
    two = ref.get_gain_tau(True).as_dict()
    assert ref.launch_count == 4
    ref.close()

    # statistics asked for between the two halves: completed by the one-block kernel, then a plain update
    ada = B.AdaScale(numels, 8, **kw)
    w, v = [t.clone() for t in w0], [t.clone() for t in v0]
    ada.reduce(rows, sched)
    assert ada.get_gain_tau(True).as_dict() == one
    assert ada.launch_count == 2
    ada.update(w, v)
    ada.update(w, v)        # a second update reads eta_t from the state and applies it once more
    torch.cuda.synchronize()
    assert ada.launch_count == 4
    assert ada.get_gain_tau(True).as_dict() == one
    ada.close()

    ada = B.AdaScale(numels, 8, **kw)
    w, v = [t.clone() for t in w0], [t.clone() for t in v0]
    ada.reduce(rows, sched)
    assert ada.get_gain_tau(True).t == 1
    ada.update(w, v)
    torch.cuda.synchronize()
    for a, b in zip(w + v, w_one + v_one):
        assert torch.equal(a, b)
    ada.close()

    # two reduce calls in a row: the first iteration is completed before the second starts
    ada = B.AdaScale(numels, 8, **kw)
    ada.reduce(rows, sched)
    ada.reduce(rows2, sched)
    assert ada.get_gain_tau(True).as_dict() == two
    assert ada.launch_count == 4      # reduce, scalar, reduce, scalar
    ada.close()

    # a state set from outside replaces everything, an open iteration included
    donor = B.AdaScale(numels, 8, **kw)
    blob = donor.get_state()
    donor.close()
    ada = B.AdaScale(numels, 8, **kw)
    ada.reduce(rows, sched)
    ada.set_state(blob)
    st = ada.get_gain_tau(True)
    assert st.t == 0 and st.tau == 0.0
    ada.reduce(rows, sched)
    assert ada.get_gain_tau(True).as_dict()["r"] == one["r"]
    ada.close()


def test_the_open_scalar_part_and_the_last_block_form_agree():
    """Runs from the counter keep the scalar part in the reduce kernel's last block; the static
    assignment leaves it to the update kernel.  Same functions, sums in a different order."""
    numels, rows, w0, v0 = _open_job(79, S=16)
    sched = B.make_schedule("exp", eta0=0.1, d=0.5, T_S1=4.0)
    out = []
    for runs in (0, 2):
        ada = B.AdaScale(numels, 16, momentum=0.9)
        ada.set_tile_runs(runs)
        w, v = [t.clone() for t in w0], [t.clone() for t in v0]
        for _ in range(3):
            ada.step(rows, w, v, sched)
        out.append((ada.get_gain_tau(True), w, v))
        ada.close()
    a, b = out[0][0], out[1][0]
    for f in ("r", "tau", "eta", "sigma2_raw", "mu2_raw", "sigma2_avg", "mu2_avg"):
        assert abs(getattr(a, f) - getattr(b, f)) <= 1e-12 * abs(getattr(b, f)), f
    assert a.t == b.t == 3
    for x, y in zip(out[0][1] + out[0][2], out[1][1] + out[1][2]):
        assert torch.allclose(x, y, rtol=1e-6, atol=1e-7)


def test_large_job_form_with_the_pair_sum_kernel():
    """Runs from the counter in the two-kernel form: reduce, a small kernel that adds up the run pairs, update
    (three launches per step); a reduce call that no update follows is completed by the one-block kernel."""
    numels, rows, w0, v0 = _open_job(81, S=16)
    sched = B.make_schedule("const", eta0=0.05)
    ref = B.AdaScale(numels, 16, momentum=0.9)
    ref.set_tile_runs(2)
    w, v = [t.clone() for t in w0], [t.clone() for t in v0]
    ref.step(rows, w, v, sched)
    torch.cuda.synchronize()
    assert ref.launch_count == 3
    one = ref.get_gain_tau(True).as_dict()
    ref.close()

    ada = B.AdaScale(numels, 16, momentum=0.9)
    ada.set_tile_runs(2)
    w2, v2 = [t.clone() for t in w0], [t.clone() for t in v0]
    ada.reduce(rows, sched)
    assert ada.get_gain_tau(True).as_dict() == one
    assert ada.launch_count == 3       # reduce, pair sum, scalar
    ada.update(w2, v2)
    torch.cuda.synchronize()
    for a, b in zip(w + v, w2 + v2):
        assert torch.equal(a, b)
    ada.close()
