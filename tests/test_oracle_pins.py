"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests re-types the oracle's own loop: each compares it with an
independent statement (exact rational arithmetic of the formula as the paper
prints it, numpy's sample variance, closed forms, the paper's fixed points).
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _rows(rng, S, P, mean_scale=1.0, noise=1.0):
    m = rng.normal(0.0, mean_scale, P)
    return [(m + noise * rng.normal(0.0, 1.0, P)).astype(np.float32) for _ in range(S)]


def _paper_formulas_exact(rows):
    """App. B.3 exactly as printed, in rational arithmetic."""
    S = len(rows)
    P = rows[0].size
    fr = [[Fraction(float(x)) for x in row] for row in rows]
    Q = sum(x * x for row in fr for x in row)
    gbar = [sum(fr[i][j] for i in range(S)) / S for j in range(P)]
    N = sum(x * x for x in gbar)
    sigma2 = Fraction(1, S - 1) * Q - Fraction(S, S - 1) * N
    mu2 = N - sigma2 / S
    return sigma2, mu2, Q, N, gbar


# ----------------------------------------------------------------- estimates


@pytest.mark.parametrize("S,P", [(2, 1), (2, 5), (3, 4), (5, 7), (8, 3), (7, 16)])
def test_estimates_match_printed_formula_in_rational_arithmetic(oracle_mod, S, P):
    rng = np.random.default_rng(100 * S + P)
    rows = _rows(rng, S, P)
    sigma2, mu2, Q, N, gbar = _paper_formulas_exact(rows)
    g, D, Nn, Qq = oracle_mod.grad_stats(rows)
    assert Qq == pytest.approx(float(Q), rel=1e-13)
    assert Nn == pytest.approx(float(N), rel=1e-13)
    assert D / (S - 1) == pytest.approx(float(sigma2), rel=1e-12)
    np.testing.assert_allclose(g, [float(x) for x in gbar], rtol=1e-15)
    orc = oracle_mod.Oracle(S, theta=0.0, eps=0.0)
    orc.reduce([[r] for r in rows])
    st = orc.scalar(oracle_mod.make_lr())
    assert st["sigma2_raw"] == pytest.approx(float(sigma2), rel=1e-12)
    assert st["mu2_raw"] == pytest.approx(float(mu2), rel=1e-11, abs=1e-13 * float(Q))
    # algebraic equivalence with the estimator of Sec. 3.4
    assert st["sigma2_raw"] + st["mu2_raw"] == pytest.approx(float(Q) / S, rel=1e-12)
    assert st["sigma2_raw"] / S + st["mu2_raw"] == pytest.approx(float(N), rel=1e-12)


@pytest.mark.parametrize("S", [2, 3, 4, 8])
def test_sigma2_is_summed_per_coordinate_sample_variance(oracle_mod, S):
    rng = np.random.default_rng(S)
    rows = _rows(rng, S, 64)
    _, D, _, _ = oracle_mod.grad_stats(rows)
    G = np.stack(rows).astype(np.float64)
    assert D / (S - 1) == pytest.approx(np.var(G, axis=0, ddof=1).sum(), rel=1e-13)
    # and with extended precision
    Gl = G.astype(np.longdouble)
    dev = ((Gl - Gl.mean(axis=0)) ** 2).sum()
    assert D == pytest.approx(float(dev), rel=1e-13)


def test_gain_theta0_equals_ratio_of_norms(oracle_mod):
    """theta = 0, no clamp active: r = ((1/S) sum ||g_i||^2) / ||gbar||^2 (Sec. 3.4)."""
    rng = np.random.default_rng(7)
    for S, P in [(2, 9), (4, 33), (6, 5)]:
        rows = _rows(rng, S, P, mean_scale=2.0, noise=0.5)
        _, _, Q, N, _ = _paper_formulas_exact(rows)
        orc = oracle_mod.Oracle(S, theta=0.0, eps=0.0)
        orc.reduce([[r] for r in rows])
        st = orc.scalar(oracle_mod.make_lr())
        assert st["mu2_raw"] > 0 and st["sigma2_raw"] > 0
        assert st["r"] == pytest.approx(float(Q / S / N), rel=1e-12)
        # the recommended estimator with eps = 0 is the same number
        orc2 = oracle_mod.Oracle(S, theta=0.0, eps=0.0, flags=oracle_mod.FLAG_RATIO)
        orc2.reduce([[r] for r in rows])
        assert orc2.scalar(oracle_mod.make_lr())["r"] == pytest.approx(st["r"], rel=1e-12)


def test_ratio_estimator_eps(oracle_mod):
    rows = [np.array([3.0, 4.0], np.float32), np.array([1.0, 0.0], np.float32)]
    # (1/S) sum ||g||^2 = (25 + 1)/2 = 13; gbar = (2, 2), ||gbar||^2 = 8
    orc = oracle_mod.Oracle(2, theta=0.0, eps=0.5, flags=oracle_mod.FLAG_RATIO)
    orc.reduce([[r] for r in rows])
    assert orc.scalar(oracle_mod.make_lr())["r"] == pytest.approx(13.5 / 8.5, rel=1e-15)


def test_hand_worked_example(oracle_mod):
    """S = 2, P = 2, values chosen so everything is a small integer."""
    rows = [np.array([3.0, 1.0], np.float32), np.array([1.0, 3.0], np.float32)]
    # gbar = (2, 2); N = 8; Q = 20; sigma^2 = 20 - 2*8 = 4; mu^2 = 8 - 2 = 6
    # r = (4 + 6) / (4/2 + 6) = 1.25
    orc = oracle_mod.Oracle(2, theta=0.0, momentum=0.5, weight_decay=0.25)
    w = [np.array([4.0, -8.0])]
    v = [np.array([2.0, 0.0])]
    st = orc.step([[r] for r in rows], w, v, oracle_mod.make_lr("const", eta0=0.5))
    assert st["sigma2_raw"] == 4.0 and st["mu2_raw"] == 6.0 and st["r"] == 1.25
    assert st["eta"] == 0.625 and st["tau"] == 1.25
    # v = 0.5*(2, 0) + (2, 2) + 0.25*(4, -8) = (4, 0); w = (4, -8) - 0.625*(4, 0)
    np.testing.assert_array_equal(v[0], [4.0, 0.0])
    np.testing.assert_array_equal(w[0], [1.5, -8.0])


# -------------------------------------------------------------- fixed points


@pytest.mark.parametrize("S", [2, 4, 8, 16])
def test_identical_rows_give_zero_variance_and_unit_gain(oracle_mod, S):
    rng = np.random.default_rng(S)
    row = rng.normal(0, 1, 257).astype(np.float32)
    orc = oracle_mod.Oracle(S, theta=0.0)
    D, N, _ = orc.reduce([[row.copy()] for _ in range(S)])
    assert D == 0.0
    st = orc.scalar(oracle_mod.make_lr())
    assert st["sigma2_raw"] == 0.0 and st["sigma2_hat"] == 1e-6
    bound = 1e-6 * (1 - 1 / S) / N
    assert 1.0 <= st["r"] <= 1.0 + 1.01 * bound


@pytest.mark.parametrize("S", [2, 8, 32])
def test_zero_mean_noise_gives_gain_near_S(oracle_mod, S):
    rng = np.random.default_rng(S)
    P = 20000
    rows = [rng.normal(0, 1, P).astype(np.float32) for _ in range(S)]
    orc = oracle_mod.Oracle(S, theta=0.0)
    orc.reduce([[r] for r in rows])
    r = orc.scalar(oracle_mod.make_lr())["r"]
    assert r <= S
    assert r >= S * (1 - 6 * S / math.sqrt(P))


@pytest.mark.parametrize("S,k", [(4, 10.0), (8, 0.3), (8, 3.0), (8, 30.0), (16, 3.0)])
def test_statistical_closed_form(oracle_mod, S, k):
    """E r ~ (k^2+1)/(k^2/S+1) for g_i = m + s n_i with k = s/std(m) (Eq. 3)."""
    rng = np.random.default_rng(11)
    P = 200000
    m = rng.normal(0, 0.1, P)
    rows = [(m + 0.1 * k * rng.normal(0, 1, P)).astype(np.float32) for _ in range(S)]
    orc = oracle_mod.Oracle(S, theta=0.0)
    orc.reduce([[r] for r in rows])
    r = orc.scalar(oracle_mod.make_lr())["r"]
    expect = (k * k + 1) / (k * k / S + 1)
    assert r == pytest.approx(expect, rel=0.03)


def test_estimators_are_unbiased(oracle_mod):
    rng = np.random.default_rng(5)
    S, P, s = 4, 50, 0.7
    m = rng.normal(0, 1, P)
    sig, mu = [], []
    for _ in range(4000):
        rows = [(m + s * rng.normal(0, 1, P)).astype(np.float32) for _ in range(S)]
        orc = oracle_mod.Oracle(S, theta=0.0)
        orc.reduce([[r] for r in rows])
        st = orc.scalar(oracle_mod.make_lr())
        sig.append(st["sigma2_raw"])
        mu.append(st["mu2_raw"])
    true_sigma2, true_mu2 = P * s * s, float((m * m).sum())
    assert np.mean(sig) == pytest.approx(true_sigma2, abs=5 * np.std(sig) / math.sqrt(len(sig)))
    assert np.mean(mu) == pytest.approx(true_mu2, abs=5 * np.std(mu) / math.sqrt(len(mu)))


def test_scale_one_has_unit_gain(oracle_mod):
    rng = np.random.default_rng(1)
    orc = oracle_mod.Oracle(1)
    for t in range(5):
        st = orc.step([[rng.normal(0, 1, 10).astype(np.float32)]], [np.zeros(10)], [np.zeros(10)],
                      oracle_mod.make_lr())
        assert st["r"] == 1.0 and st["tau"] == t + 1


def test_gain_stays_in_range_on_adversarial_scales(oracle_mod):
    rng = np.random.default_rng(3)
    for trial in range(300):
        S = int(rng.integers(2, 12))
        P = int(rng.integers(1, 40))
        scale = 10.0 ** rng.uniform(-12, 8)
        rows = _rows(rng, S, P, mean_scale=scale * 10.0 ** rng.uniform(-3, 3), noise=scale)
        orc = oracle_mod.Oracle(S, theta=float(rng.choice([0.0, 0.5, -1.0])))
        for _ in range(3):
            orc.reduce([[r] for r in rows])
            r = orc.scalar(oracle_mod.make_lr())["r"]
            assert 1.0 <= r <= S * (1 + 1e-12)


def test_all_zero_gradients(oracle_mod):
    orc = oracle_mod.Oracle(4)
    orc.reduce([[np.zeros(8, np.float32)] for _ in range(4)])
    st = orc.scalar(oracle_mod.make_lr())
    assert st["sigma2_hat"] == 1e-6 and st["mu2_hat"] == 0.0 and st["r"] == 4.0


# -------------------------------------------------------------- clock, averages


def test_tau_accumulates_the_gains(oracle_mod):
    rng = np.random.default_rng(9)
    S = 8
    orc = oracle_mod.Oracle(S)
    total, T_SI, iters = 0.0, 200.0, 0
    while orc.state.tau < T_SI:
        rows = _rows(rng, S, 50, mean_scale=0.3, noise=1.0)
        orc.reduce([[r] for r in rows])
        st = orc.scalar(oracle_mod.make_lr())
        total += st["r"]
        iters += 1
        assert st["tau"] == pytest.approx(total, rel=1e-15)
        assert st["t"] == iters
    assert math.ceil(T_SI / S) <= iters <= T_SI


def test_theta_rule(oracle_mod):
    assert oracle_mod.Oracle(16).theta == pytest.approx(1 - 16 / 1000)
    assert oracle_mod.Oracle(999).theta == pytest.approx(0.001)
    assert oracle_mod.Oracle(1000).theta == 0.0
    assert oracle_mod.Oracle(4096).theta == 0.0
    assert oracle_mod.Oracle(16, theta=0.25).theta == 0.25


def _feed(orc, oracle_mod, sigma2, mu2, lr=None):
    """S = 2: D = sigma2, N = mu2 + sigma2 / 2 produce exactly these estimates."""
    lr = oracle_mod.make_lr() if lr is None else lr
    return orc.scalar(lr, D=sigma2, N=mu2 + sigma2 / 2.0, Q=0.0)


def test_average_is_plain_mean_during_warm_up_then_geometric(oracle_mod):
    theta = 0.9  # hand-over at n = 1/(1-theta) = 10
    orc = oracle_mod.Oracle(2, theta=theta)
    for n in range(1, 10):
        st = _feed(orc, oracle_mod, float(n), 2.0 * n)
        assert st["avg_a"] == pytest.approx((n + 1) / 2, rel=1e-14)
        assert st["avg_b"] == pytest.approx(n + 1.0, rel=1e-14)
    a0 = orc.state.avg_a
    # from now on a constant input b is approached geometrically: b + (a0 - b) theta^k
    for k in range(1, 30):
        st = _feed(orc, oracle_mod, 100.0, 7.0)
        assert st["avg_a"] == pytest.approx(100.0 + (a0 - 100.0) * theta ** k, rel=1e-12)


def test_constant_samples_keep_constant_average_and_theta0_means_no_average(oracle_mod):
    orc = oracle_mod.Oracle(2, theta=0.95)
    for _ in range(60):
        st = _feed(orc, oracle_mod, 3.0, 5.0)
        assert st["avg_a"] == pytest.approx(3.0, rel=1e-14) and st["avg_b"] == pytest.approx(5.0, rel=1e-14)
    orc = oracle_mod.Oracle(2, theta=0.0)
    for n in range(1, 6):
        st = _feed(orc, oracle_mod, float(n), 1.0)
        assert st["avg_a"] == float(n)


def test_clamps_apply_before_averaging(oracle_mod):
    orc = oracle_mod.Oracle(2, theta=0.5, eps=1e-3)
    st = orc.scalar(oracle_mod.make_lr(), D=0.0, N=4.0, Q=0.0)
    assert st["sigma2_hat"] == 1e-3 and st["avg_a"] == 1e-3
    # negative raw mu^2 is clamped at zero; it is built from the unclamped sigma^2
    st = orc.scalar(oracle_mod.make_lr(), D=10.0, N=1.0, Q=0.0)
    assert st["mu2_raw"] == -4.0 and st["mu2_hat"] == 0.0
    assert st["avg_b"] == pytest.approx(0.5 * 4.0 + 0.5 * 0.0)


def test_lagged_mode_uses_prior_iterations_only(oracle_mod):
    rng = np.random.default_rng(2)
    S = 4
    cur = oracle_mod.Oracle(S, theta=0.8)
    lag = oracle_mod.Oracle(S, theta=0.8, flags=oracle_mod.FLAG_LAGGED)
    prev = 1.0  # r_0 = 1
    for _ in range(12):
        rows = _rows(rng, S, 30)
        for o in (cur, lag):
            o.reduce([[r] for r in rows])
        rc = cur.scalar(oracle_mod.make_lr())["r"]
        rl = lag.scalar(oracle_mod.make_lr())["r"]
        assert rl == prev
        prev = rc


def test_lagged_ratio_estimator_uses_prior_iterations_only(oracle_mod):
    """Sec. 3.4's estimator with App. B.3's lag: r_0 = 1, then the current-mode ratio gain of the iteration before."""
    rng = np.random.default_rng(12)
    S = 4
    flags = oracle_mod.FLAG_RATIO
    cur = oracle_mod.Oracle(S, theta=0.8, eps=0.25, flags=flags)
    lag = oracle_mod.Oracle(S, theta=0.8, eps=0.25, flags=flags | oracle_mod.FLAG_LAGGED)
    prev = 1.0  # r_0 = 1
    taus = 0.0
    for _ in range(12):
        rows = _rows(rng, S, 30)
        for o in (cur, lag):
            o.reduce([[r] for r in rows])
        rc = cur.scalar(oracle_mod.make_lr())["r"]
        sl = lag.scalar(oracle_mod.make_lr())
        assert sl["r"] == prev
        taus += prev
        assert sl["tau"] == pytest.approx(taus, rel=1e-15)
        # both modes keep the same averages: only the gain that is read out lags
        assert sl["avg_a"] == cur.state.avg_a and sl["avg_b"] == cur.state.avg_b
        prev = rc


def test_lagged_ratio_estimator_hand_worked(oracle_mod):
    """Three iterations by hand, S = 2, theta = 1/2, eps = 1/2 (every value a dyadic rational).

    m1 averages (1/S) sum_i ||g_i||^2, m2 averages ||gbar||^2, r = (m1 + eps) / (m2 + eps)   (Sec. 3.4),
    read from the averages of prior iterations only, r_0 = 1   (App. B.3).
    """
    orc = oracle_mod.Oracle(2, theta=0.5, eps=0.5, flags=oracle_mod.FLAG_RATIO | oracle_mod.FLAG_LAGGED)
    lr = oracle_mod.make_lr("const", eta0=2.0)
    # iteration 0: samples (13, 8); no prior average -> r = 1; averages become (13, 8)
    orc.reduce([[np.array([3.0, 4.0], np.float32)], [np.array([1.0, 0.0], np.float32)]])
    st = orc.scalar(lr)
    assert st["r"] == 1.0 and st["eta"] == 2.0 and st["tau"] == 1.0
    assert (st["avg_a"], st["avg_b"]) == (13.0, 8.0)
    # iteration 1: samples (2, 1); r from the prior averages = 13.5 / 8.5; the second sample is
    # still inside the plain-mean warm-up: averages ((13 + 2)/2, (8 + 1)/2) = (7.5, 4.5)
    orc.reduce([[np.array([1.0, 1.0], np.float32)], [np.array([1.0, -1.0], np.float32)]])
    st = orc.scalar(lr)
    assert st["r"] == pytest.approx(13.5 / 8.5, rel=1e-15)
    assert st["eta"] == pytest.approx(27.0 / 8.5, rel=1e-15)
    assert (st["avg_a"], st["avg_b"]) == (7.5, 4.5)
    # iteration 2: r = (7.5 + 0.5) / (4.5 + 0.5) = 1.6 whatever this iteration's gradients are;
    # samples (8, 8) enter with weight 1 - theta: averages (7.75, 6.25)
    orc.reduce([[np.array([2.0, 2.0], np.float32)], [np.array([2.0, 2.0], np.float32)]])
    st = orc.scalar(lr)
    assert st["r"] == pytest.approx(1.6, rel=1e-15)
    assert st["tau"] == pytest.approx(1.0 + 13.5 / 8.5 + 1.6, rel=1e-15)
    assert (st["avg_a"], st["avg_b"]) == (7.75, 6.25)


def test_elastic_scale_change_keeps_averages(oracle_mod):
    orc = oracle_mod.Oracle(2, theta=0.5)
    _feed(orc, oracle_mod, 4.0, 6.0)
    orc.set_scale(4)
    # S = 4 now: sigma^2 = D/3, mu^2 = N - sigma^2/4
    st = orc.scalar(oracle_mod.make_lr(), D=12.0, N=7.0, Q=0.0)
    assert st["sigma2_raw"] == 4.0 and st["mu2_raw"] == 6.0
    assert st["r"] == pytest.approx((4.0 + 6.0) / (4.0 / 4 + 6.0))


def test_nonfinite_sums_skip_the_step(oracle_mod):
    orc = oracle_mod.Oracle(2, theta=0.5)
    _feed(orc, oracle_mod, 4.0, 6.0)
    before = (orc.state.tau, orc.state.avg_a, orc.state.avg_b, orc.state.n, orc.state.t)
    rows = [np.array([1.0, np.inf], np.float32), np.array([1.0, 2.0], np.float32)]
    w, v = [np.ones(2)], [np.ones(2)]
    st = orc.step([[r] for r in rows], w, v, oracle_mod.make_lr())
    assert st["nonfinite"] == 1 and st["eta"] == 0.0 and st["skipped"] == 1
    assert before == (orc.state.tau, orc.state.avg_a, orc.state.avg_b, orc.state.n, orc.state.t)
    np.testing.assert_array_equal(w[0], 1.0)
    np.testing.assert_array_equal(v[0], 1.0)


# -------------------------------------------------------------- schedules


def _golden_rows():
    with open(os.path.join(GOLDEN, "lr_table3.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                yield line.split()


def test_lr_schedules_of_table3(oracle_mod):
    n = 0
    for name, fam, eta0, d, T, ws, t, expect in _golden_rows():
        ms = () if ws == "-" else tuple(float(x) for x in ws.split(","))
        lr = oracle_mod.make_lr(fam, eta0=float(eta0), d=float(d), T_S1=1.0 if T == "-" else float(T),
                                milestones=ms)
        assert oracle_mod.lr_eval(lr, float(t)) == pytest.approx(float(expect), rel=1e-13), (name, t)
        n += 1
    assert n >= 20


def test_lr_is_read_at_floor_of_tau(oracle_mod):
    lr = oracle_mod.make_lr("step", eta0=1.0, d=0.5, milestones=(2.0,))
    orc = oracle_mod.Oracle(2, theta=0.0)
    # gains: sigma^2 = mu^2 -> r = 2/(1.5) = 4/3 ; tau = 0, 4/3, 8/3, 4
    seen = []
    for _ in range(4):
        st = _feed(orc, oracle_mod, 1.0, 1.0, lr)
        seen.append(st["lr"])
    # floor(tau) = 0, 1, 2, 4 -> only the last exceeds the boundary 2 (strict)
    assert seen == [1.0, 1.0, 1.0, 0.5]
    orc = oracle_mod.Oracle(2, theta=0.0, flags=oracle_mod.FLAG_CONT_TAU)
    seen = [_feed(orc, oracle_mod, 1.0, 1.0, lr)["lr"] for _ in range(4)]
    assert seen == [1.0, 1.0, 0.5, 0.5]  # tau = 8/3 > 2 already


# -------------------------------------------------------------- update


def test_update_without_momentum_is_eq2(oracle_mod):
    rng = np.random.default_rng(4)
    S, P = 4, 37
    rows = _rows(rng, S, P)
    w0 = rng.normal(0, 1, P)
    w, v = [w0.copy()], [np.zeros(P)]
    orc = oracle_mod.Oracle(S, theta=0.0)
    st = orc.step([[r] for r in rows], w, v, oracle_mod.make_lr("const", eta0=0.3))
    gbar = np.mean(np.stack(rows).astype(np.float64), axis=0)
    np.testing.assert_allclose(w[0], w0 - st["eta"] * gbar, rtol=1e-14, atol=1e-16)
    assert st["eta"] == pytest.approx(st["r"] * 0.3, rel=1e-15)


def test_momentum_geometric_series(oracle_mod):
    """Constant gradient g, constant eta: v_t = g (1-rho^t)/(1-rho), w_t = w_0 - eta sum_k v_k."""
    rho, eta = 0.9, 0.05
    g = np.array([1.0, -2.0, 0.5], np.float32)
    orc = oracle_mod.Oracle(1, momentum=rho)
    w, v = [np.array([1.0, 1.0, 1.0])], [np.zeros(3)]
    acc = 0.0
    for t in range(1, 40):
        orc.step([[g]], w, v, oracle_mod.make_lr("const", eta0=eta))
        geo = (1 - rho ** t) / (1 - rho)
        acc += geo
        np.testing.assert_allclose(v[0], g.astype(np.float64) * geo, rtol=1e-13)
        np.testing.assert_allclose(w[0], 1.0 - eta * acc * g.astype(np.float64), rtol=1e-12)


def test_weight_decay_fixed_point(oracle_mod):
    """g = -lambda w makes gbar + lambda w vanish: with v = 0 nothing moves."""
    lam = 0.25  # exact in binary, so g = -lambda w is exact in float32
    w0 = np.array([2.0, -4.0, 8.0])
    g = (-lam * w0).astype(np.float32)
    w, v = [w0.copy()], [np.zeros(3)]
    orc = oracle_mod.Oracle(1, momentum=0.9, weight_decay=lam)
    orc.step([[g]], w, v, oracle_mod.make_lr())
    np.testing.assert_array_equal(v[0], 0.0)
    np.testing.assert_array_equal(w[0], w0)


# -------------------------------------------------------------- inputs, threads


def test_bf16_bits_are_upcast_exactly(oracle_mod):
    import torch
    bits = np.arange(65536, dtype=np.int64)
    finite = bits[((bits >> 7) & 0xFF) != 0xFF].astype(np.uint16)
    ref = torch.from_numpy(finite.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    g, _, _, _ = oracle_mod.grad_stats([finite])
    np.testing.assert_array_equal(g, ref)


def test_threads_do_not_change_the_result(oracle_mod):
    rng = np.random.default_rng(6)
    rows = _rows(rng, 5, 100003)
    g1, D1, N1, Q1 = oracle_mod.grad_stats(rows, nthreads=1)
    g4, D4, N4, Q4 = oracle_mod.grad_stats(rows, nthreads=4)
    np.testing.assert_array_equal(g1, g4)
    assert D4 == pytest.approx(D1, rel=1e-13) and N4 == pytest.approx(N1, rel=1e-13)
    assert Q4 == pytest.approx(Q1, rel=1e-13)


def test_multi_tensor_equals_concatenation(oracle_mod):
    rng = np.random.default_rng(8)
    S, sizes = 3, [1, 5, 64, 7]
    parts = [[rng.normal(0, 1, n).astype(np.float32) for n in sizes] for _ in range(S)]
    a = oracle_mod.Oracle(S, theta=0.0)
    a.reduce(parts)
    b = oracle_mod.Oracle(S, theta=0.0)
    b.reduce([[np.concatenate(p)] for p in parts])
    assert a.D == pytest.approx(b.D, rel=1e-14) and a.N == pytest.approx(b.N, rel=1e-14)
