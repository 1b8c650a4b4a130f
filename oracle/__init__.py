"""ctypes access to the AdaScale CPU oracle (``adascale_oracle.c``).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this package.  It imports nothing from
the CUDA package and the CUDA package imports nothing from here.

The arithmetic lives in the C file; this module only builds it with gcc, lays
out the structs and walks the tensor list.  Gradients are numpy arrays of
``float32`` or, for bf16, ``uint16`` holding the raw bf16 bits; parameters and
momentum are ``float64`` arrays that the oracle updates in place.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# The mutation test points this at a deliberately broken copy of the C file.
_SRC = os.environ.get("ADASCALE_ORACLE_SRC", os.path.join(_HERE, "adascale_oracle.c"))
_LIB = os.path.join(_HERE, "liboracle.so") if "ADASCALE_ORACLE_SRC" not in os.environ else _SRC + ".so"

F32, BF16 = 0, 1
LR_CONST, LR_EXP, LR_STEP = 0, 1, 2
FLAG_LAGGED, FLAG_CONT_TAU, FLAG_RATIO = 1, 2, 4


class LR(C.Structure):
    _fields_ = [("kind", C.c_int), ("eta0", C.c_double), ("d", C.c_double), ("T_S1", C.c_double),
                ("n", C.c_int), ("w", C.c_double * 8)]


class Cfg(C.Structure):
    _fields_ = [("S", C.c_int), ("eps", C.c_double), ("theta", C.c_double), ("flags", C.c_int)]


class State(C.Structure):
    _fields_ = [("tau", C.c_double), ("avg_a", C.c_double), ("avg_b", C.c_double),
                ("n", C.c_longlong), ("t", C.c_longlong), ("skipped", C.c_longlong),
                ("r", C.c_double), ("eta", C.c_double), ("lr", C.c_double),
                ("sigma2_raw", C.c_double), ("mu2_raw", C.c_double),
                ("sigma2_hat", C.c_double), ("mu2_hat", C.c_double), ("nonfinite", C.c_int)]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (strict fp64: no fast-math) and return the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.oracle_lr_eval.restype = C.c_double
        L.oracle_lr_eval.argtypes = [C.POINTER(LR), C.c_double]
        L.oracle_theta.restype = C.c_double
        L.oracle_theta.argtypes = [C.POINTER(Cfg)]
        L.oracle_grad_stats.restype = None
        L.oracle_grad_stats.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_longlong, C.c_int, C.c_void_p,
                                        C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_double),
                                        C.c_int]
        L.oracle_scalar_step.restype = None
        L.oracle_scalar_step.argtypes = [C.POINTER(State), C.POINTER(Cfg), C.POINTER(LR), C.c_double,
                                         C.c_double, C.c_double]
        L.oracle_update.restype = None
        L.oracle_update.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_longlong, C.c_double,
                                    C.c_double, C.c_double, C.c_int]
        _lib = L
    return _lib


def make_lr(kind="const", eta0=0.1, d=1.0, T_S1=1.0, milestones=()):
    kinds = {"const": LR_CONST, "exp": LR_EXP, "step": LR_STEP}
    s = LR()
    s.kind = kinds[kind]
    s.eta0, s.d, s.T_S1 = float(eta0), float(d), float(T_S1)
    s.n = len(milestones)
    for i, m in enumerate(milestones):
        s.w[i] = float(m)
    return s


def lr_eval(lr: LR, t: float) -> float:
    return lib().oracle_lr_eval(C.byref(lr), float(t))


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError("gradient rows are float32 or uint16 (raw bf16 bits), got %s" % a.dtype)


def grad_stats(rows, want_gbar=True, nthreads=1):
    """rows: S equally long 1-D arrays.  Returns (gbar float64 or None, D, N, Q)."""
    S = len(rows)
    n = rows[0].size
    code = _dtype_code(rows[0])
    for a in rows:
        assert a.size == n and _dtype_code(a) == code and a.flags.c_contiguous
    ptrs = (C.c_void_p * S)(*[a.ctypes.data for a in rows])
    gbar = np.empty(n, dtype=np.float64) if want_gbar else None
    D, N, Q = C.c_double(0.0), C.c_double(0.0), C.c_double(0.0)
    lib().oracle_grad_stats(ptrs, S, n, code, gbar.ctypes.data if want_gbar else None, C.byref(D),
                            C.byref(N), C.byref(Q), int(nthreads))
    return gbar, D.value, N.value, Q.value


class Oracle:
    """State of one AdaScale run plus the walk over the tensor list."""

    def __init__(self, S, momentum=0.0, weight_decay=0.0, eps=1e-6, theta=-1.0, flags=0, nthreads=1):
        self.cfg = Cfg(int(S), float(eps), float(theta), int(flags))
        self.rho = float(momentum)
        self.lam = float(weight_decay)
        self.state = State()
        self.nthreads = int(nthreads)
        self.gbar = None
        self.D = self.N = self.Q = 0.0

    @property
    def theta(self):
        return lib().oracle_theta(C.byref(self.cfg))

    def set_scale(self, S):
        """Elastic scaling: S changes between iterations, the averages carry over."""
        self.cfg.S = int(S)

    def reduce(self, grads):
        """grads[i][k]: row i, tensor k.  Accumulates D, N, Q over all tensors."""
        S = self.cfg.S
        assert len(grads) == S
        T = len(grads[0])
        self.D = self.N = self.Q = 0.0
        self.gbar = []
        for k in range(T):
            g, D, N, Q = grad_stats([grads[i][k].reshape(-1) for i in range(S)], True, self.nthreads)
            self.gbar.append(g)
            self.D += D
            self.N += N
            self.Q += Q
        return self.D, self.N, self.Q

    def scalar(self, lr, D=None, N=None, Q=None):
        D = self.D if D is None else D
        N = self.N if N is None else N
        Q = self.Q if Q is None else Q
        lib().oracle_scalar_step(C.byref(self.state), C.byref(self.cfg), C.byref(lr), D, N, Q)
        return self.stats()

    def update(self, w, v, gbar=None):
        gbar = self.gbar if gbar is None else gbar
        if self.state.nonfinite:
            return
        for k in range(len(w)):
            assert w[k].dtype == np.float64 and v[k].dtype == np.float64
            lib().oracle_update(gbar[k].ctypes.data, w[k].ctypes.data, v[k].ctypes.data, w[k].size,
                                self.rho, self.lam, self.state.eta, self.nthreads)

    def step(self, grads, w, v, lr):
        """One whole iteration in the paper's order; returns the step's scalars."""
        self.reduce(grads)
        out = self.scalar(lr)
        self.update(w, v)
        return out

    def stats(self):
        s = self.state
        return {"r": s.r, "tau": s.tau, "eta": s.eta, "lr": s.lr, "sigma2_raw": s.sigma2_raw,
                "mu2_raw": s.mu2_raw, "sigma2_hat": s.sigma2_hat, "mu2_hat": s.mu2_hat,
                "avg_a": s.avg_a, "avg_b": s.avg_b, "n": s.n, "t": s.t, "skipped": s.skipped,
                "nonfinite": s.nonfinite, "gbar_sqnorm": self.N}
