"""Shared by the GPU parity tests: runs the CUDA library and the CPU oracle on the same bytes."""
import os

import numpy as np
import torch

import oracle
from paper_2007_05105_b200 import binding as B

NTHREADS = max(1, min(32, os.cpu_count() or 1))

# Tolerances (fp32 arithmetic on the device against the fp64 oracle):
#   sigma^2, mu^2 : |d| <= 1e-5 |oracle| + 1e-12 * sum_i ||g_i||^2   (the absolute part covers
#                   sigma^2 = 0 for identical rows and mu^2 clamped at 0)
#   r, eta, lr    : 1e-5 relative;  tau: 1e-5 relative per step, 1e-4 after 1000 steps
#   gbar          : max(5, 0.75 sqrt(S)) * 2^-24 * max_i |g_ij| per element (fp32 sum of the column, one
#                   rounding of the mean; the sum's error grows like sqrt(S))
#   v             : |dv| <= 1e-6 (|v| + |gbar| + |lambda w|) + the gbar tolerance
#   w             : |dw| <= 1e-6 (|w| + |eta| (|v| + |gbar|)) + |eta| * the gbar tolerance,
#                   and ||dw|| / ||w|| <= 1e-6
REL = 1e-5


def to_numpy_rows(t: torch.Tensor) -> np.ndarray:
    """float32 -> float32 array; bf16 -> uint16 array of the raw bits (what the oracle reads)."""
    t = t.detach().contiguous().cpu()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16).reshape(-1)
    return t.numpy().reshape(-1)


def oracle_lr(spec):
    return oracle.make_lr(spec.get("kind", "const"), eta0=spec.get("eta0", 0.1), d=spec.get("d", 1.0),
                          T_S1=spec.get("T_S1", 1.0), milestones=spec.get("milestones", ()))


def device_lr(spec):
    return B.make_schedule(spec.get("kind", "const"), eta0=spec.get("eta0", 0.1), d=spec.get("d", 1.0),
                           T_S1=spec.get("T_S1", 1.0), milestones=spec.get("milestones", ()))


def check_stats(dev, orc, Q, label=""):
    """dev: Stats from the device, orc: dict from the oracle."""
    atol = 1e-12 * Q
    for a, b, name in [(dev.sigma2_raw, orc["sigma2_raw"], "sigma2"), (dev.mu2_raw, orc["mu2_raw"], "mu2")]:
        assert abs(a - b) <= REL * abs(b) + atol, "%s %s: device %r oracle %r" % (label, name, a, b)
    for a, b, name in [(dev.r, orc["r"], "r"), (dev.eta, orc["eta"], "eta"), (dev.lr, orc["lr"], "lr"),
                       (dev.tau, orc["tau"], "tau"), (dev.sigma2_avg, orc["avg_a"], "avg_a")]:
        assert abs(a - b) <= REL * abs(b), "%s %s: device %r oracle %r" % (label, name, a, b)
    assert abs(dev.mu2_avg - orc["avg_b"]) <= REL * abs(orc["avg_b"]) + atol, (label, dev.mu2_avg, orc["avg_b"])
    assert dev.t == orc["t"] and dev.n_samples == orc["n"], (label, dev.t, orc["t"], dev.n_samples, orc["n"])


GBAR_ULPS = 3e-7  # 5 * 2^-24: tolerance of the mean gradient relative to max_i |g_ij|, up to S = 44


def gbar_ulps(S):
    """The rounding error of an fp32 sum of S values grows like sqrt(S): 0.75 sqrt(S) ulps beyond S = 44."""
    return max(GBAR_ULPS, 0.75 * (S ** 0.5) * 2.0 ** -24)


def row_scale(rows_np):
    """max_i |g_ij| per column: the magnitude that the fp32 sum of a column works at."""
    scale = np.zeros(rows_np[0].shape, dtype=np.float64)
    for r in rows_np:
        vals = r if r.dtype == np.float32 else (r.astype(np.uint32) << 16).view(np.float32)
        np.maximum(scale, np.abs(vals.astype(np.float64)), out=scale)
    return scale


def check_gbar(gbar_dev, gbar_orc, scale, label="", ulps=GBAR_ULPS):
    err = np.abs(gbar_dev.astype(np.float64) - gbar_orc)
    bad = err > ulps * scale + 1e-45
    assert not bad.any(), "%s gbar: %d elements off, worst %g x tolerance" % (
        label, int(bad.sum()), float((err / (ulps * scale + 1e-45)).max()))


def check_update(w_dev, v_dev, w_orc, v_orc, gbar_orc, scale, eta, lam, label="", ulps=GBAR_ULPS):
    w_dev = w_dev.astype(np.float64)
    v_dev = v_dev.astype(np.float64)
    # v = rho v + gbar + lambda w: 1e-6 of the summands, plus the mean gradient's own fp32
    # summation error, which scales with the summed values and not with their (cancelling) mean
    tol_v = 1e-6 * (np.abs(v_orc) + np.abs(gbar_orc) + abs(lam) * np.abs(w_orc)) + ulps * scale + 1e-30
    tol_w = 1e-6 * (np.abs(w_orc) + abs(eta) * (np.abs(v_orc) + np.abs(gbar_orc))) \
        + abs(eta) * ulps * scale + 1e-30
    ev, ew = np.abs(v_dev - v_orc), np.abs(w_dev - w_orc)
    assert (ev <= tol_v).all(), "%s v: worst ratio %g" % (label, float((ev / tol_v).max()))
    assert (ew <= tol_w).all(), "%s w: worst ratio %g" % (label, float((ew / tol_w).max()))
    nw = np.linalg.norm(w_orc)
    if nw > 0:
        assert np.linalg.norm(w_dev - w_orc) / nw <= 1e-6, label


class Pair:
    """The CUDA context and the oracle, stepped side by side on the same inputs.

    Parameters and momentum are stored in float32 (the workloads say so), so the oracle
    computes each update in fp64 and rounds the result to float32, its storage type.  Before
    a step whose tensors are compared, the device buffers are overwritten with the oracle's
    state, so each comparison is one step from a common state: two free-running fp32 / fp64
    trajectories drift apart by about 1e-7 * sqrt(steps), which says nothing about a step.
    Nothing the oracle reads ever comes from the device path.
    """

    def __init__(self, numels, S, grad_dtype="f32", momentum=0.0, weight_decay=0.0, eps=1e-6, theta=-1.0,
                 flags=0, max_S=0, lr=None, tile_runs=-1):
        self.numels = list(numels)
        self.S = S
        self.lr_spec = lr or {"kind": "const", "eta0": 0.1}
        self.dev = B.AdaScale(numels, S, grad_dtype, momentum, weight_decay, eps, theta, flags, 0, max_S)
        if tile_runs >= 0:  # small jobs can take the tile hand-out of large ones
            self.dev.set_tile_runs(tile_runs)
        # the one-pass kernel is a device-side arrangement of the lagged mode: same oracle
        self.fused = bool(flags & B.FLAG_FUSED)
        self.orc = oracle.Oracle(S, momentum, weight_decay, eps, theta, flags & ~B.FLAG_FUSED, nthreads=NTHREADS)
        self.lam = weight_decay
        self.sched_dev = device_lr(self.lr_spec)
        self.sched_orc = oracle_lr(self.lr_spec)
        self.w64 = self.v64 = None

    def attach(self, w_tensors, v_tensors):
        self.w_t, self.v_t = w_tensors, v_tensors
        self.w64 = [t.detach().cpu().numpy().astype(np.float64).reshape(-1) for t in w_tensors]
        self.v64 = [t.detach().cpu().numpy().astype(np.float64).reshape(-1) for t in v_tensors]

    def _push_state(self, tensors=None):
        ks = range(len(self.numels)) if tensors is None else tensors
        for k in ks:
            self.w_t[k].copy_(torch.from_numpy(self.w64[k].astype(np.float32)).view_as(self.w_t[k]))
            self.v_t[k].copy_(torch.from_numpy(self.v64[k].astype(np.float32)).view_as(self.v_t[k]))

    def _round_state(self):
        for a in self.w64 + self.v64:
            a[:] = a.astype(np.float32)

    def step(self, grads, label="", compare_tensors=True):
        """grads[i][k] torch tensors on the GPU."""
        if compare_tensors:
            self._push_state()
        self.dev.step(grads, self.w_t, self.v_t, self.sched_dev)
        st = self.dev.get_gain_tau(True)
        rows_np = [[to_numpy_rows(g) for g in row] for row in grads]
        ost = self.orc.step(rows_np, self.w64, self.v64, self.sched_orc)
        check_stats(st, ost, self.orc.Q, label)
        if compare_tensors and not ost["nonfinite"]:
            gb = None if self.fused else self.dev.mean_grad_tensors()
            for k in range(len(self.numels)):
                lab = "%s tensor %d" % (label, k)
                scale = row_scale([row[k] for row in rows_np])
                if gb is not None:
                    check_gbar(gb[k].cpu().numpy(), self.orc.gbar[k], scale, lab, gbar_ulps(self.orc.cfg.S))
                check_update(self.w_t[k].detach().cpu().numpy().reshape(-1),
                             self.v_t[k].detach().cpu().numpy().reshape(-1),
                             self.w64[k], self.v64[k], self.orc.gbar[k], scale, ost["eta"], self.lam, lab,
                             gbar_ulps(self.orc.cfg.S))
        self._round_state()
        return st, ost

    def step_streamed(self, grads, label="", sample_tensors=None):
        """Same as step() for workloads too large to mirror on the host at once: the rows of
        one tensor at a time cross to the host, feed the oracle and are dropped again."""
        T = len(self.numels)
        check = set(range(T)) if sample_tensors is None else set(sample_tensors)
        self._push_state(sorted(check))
        self.dev.step(grads, self.w_t, self.v_t, self.sched_dev)
        st = self.dev.get_gain_tau(True)
        gb = None if self.fused else self.dev.mean_grad_tensors()
        o = self.orc
        o.D = o.N = o.Q = 0.0
        o.gbar = []
        scales = {}
        for k in range(T):
            rows_k = [to_numpy_rows(grads[i][k]) for i in range(self.S)]
            g, D, N, Q = oracle.grad_stats(rows_k, True, NTHREADS)
            o.gbar.append(g)
            o.D += D
            o.N += N
            o.Q += Q
            if k in check:
                scales[k] = row_scale(rows_k)
                if gb is not None:
                    check_gbar(gb[k].cpu().numpy(), g, scales[k], "%s tensor %d" % (label, k), gbar_ulps(self.S))
            del rows_k
        ost = o.scalar(self.sched_orc)
        o.update(self.w64, self.v64)
        check_stats(st, ost, o.Q, label)
        for k in sorted(check):
            check_update(self.w_t[k].detach().cpu().numpy().reshape(-1),
                         self.v_t[k].detach().cpu().numpy().reshape(-1),
                         self.w64[k], self.v64[k], o.gbar[k], scales[k], ost["eta"], self.lam,
                         "%s tensor %d" % (label, k), gbar_ulps(self.S))
        self._round_state()
        return st, ost

    def close(self):
        self.dev.close()
