"""Thin ctypes binding of the C-ABI library (``include/adascale.h``), same names.

Argument marshalling only: every step of the AdaScale iteration runs in the CUDA
kernels of ``libadascale_b200.so``.  There is no fallback: if the library has not
been built, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libadascale_b200.so")

OK, ERR_INVALID_ARG, ERR_ALIGNMENT, ERR_CUDA, ERR_STATE, ERR_TOO_LARGE = range(6)
F32, BF16 = 0, 1
LR_CONST, LR_EXP, LR_STEP = 0, 1, 2
FLAG_LAGGED, FLAG_CONT_TAU, FLAG_RATIO, FLAG_FUSED, FLAG_GRADS_READY = 1, 2, 4, 8, 16
STATUS_NONFINITE, STATUS_WAIT_TIMEOUT = 1, 2
MAX_MILESTONES = 8
STATE_BYTES = 128

EXPORTS = ("adascale_init", "adascale_step", "adascale_reduce", "adascale_update", "adascale_reduce_sums",
           "adascale_apply_sums", "adascale_get_gain_tau",
           "adascale_mean_grad", "adascale_set_scale", "adascale_set_wait_limit", "adascale_set_tile_runs", "adascale_get_state", "adascale_set_state",
           "adascale_step_host", "adascale_stream_probe", "adascale_tiling", "adascale_grad_stats_static", "adascale_launch_count",
           "adascale_destroy",
           "adascale_strerror", "adascale_last_error")


class LrSchedule(C.Structure):
    _fields_ = [("kind", C.c_int32), ("n_milestones", C.c_int32), ("eta0", C.c_double), ("decay", C.c_double),
                ("t_s1", C.c_double), ("milestones", C.c_double * MAX_MILESTONES)]


class Config(C.Structure):
    _fields_ = [("S", C.c_int32), ("max_S", C.c_int32), ("n_tensors", C.c_int32), ("grad_dtype", C.c_int32),
                ("numel", C.POINTER(C.c_int64)), ("momentum", C.c_double), ("weight_decay", C.c_double),
                ("eps", C.c_double), ("theta", C.c_double), ("flags", C.c_uint32), ("device", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [("r", C.c_double), ("tau", C.c_double), ("eta", C.c_double), ("lr", C.c_double),
                ("sigma2_raw", C.c_double), ("mu2_raw", C.c_double), ("sigma2_avg", C.c_double),
                ("mu2_avg", C.c_double), ("gbar_sqnorm", C.c_double), ("dev_sqsum", C.c_double),
                ("t", C.c_int64), ("n_samples", C.c_int64), ("skipped", C.c_int64),
                ("status_bits", C.c_uint32), ("reserved", C.c_uint32)]

    def as_dict(self):
        return {name: getattr(self, name) for name, _ in self._fields_ if name != "reserved"}


class AdaScaleError(RuntimeError):
    def __init__(self, status, text):
        super().__init__("adascale status %d: %s" % (status, text))
        self.status = status


def _load(path=LIB_PATH):
    if not os.path.exists(path):
        raise ImportError("%s is missing: build it with `python -m paper_2007_05105_b200.build` "
                          "(there is no CPU fallback)" % path)
    L = C.CDLL(path)
    vp, vpp = C.c_void_p, C.POINTER(C.c_void_p)
    L.adascale_init.argtypes = [C.POINTER(Config), C.POINTER(vp)]
    L.adascale_step.argtypes = [vp, vpp, vpp, vpp, C.POINTER(LrSchedule), vp]
    L.adascale_reduce.argtypes = [vp, vpp, C.POINTER(LrSchedule), vp]
    L.adascale_update.argtypes = [vp, vpp, vpp, vp]
    L.adascale_reduce_sums.argtypes = [vp, vpp, vp, vp]
    L.adascale_apply_sums.argtypes = [vp, vp, C.POINTER(LrSchedule), vpp, vpp, vp]
    L.adascale_get_gain_tau.argtypes = [vp, C.POINTER(Stats), C.c_int]
    L.adascale_mean_grad.argtypes = [vp, vpp]
    L.adascale_set_scale.argtypes = [vp, C.c_int32]
    L.adascale_set_wait_limit.argtypes = [vp, C.c_uint32]
    L.adascale_set_tile_runs.argtypes = [vp, C.c_int32]
    L.adascale_get_state.argtypes = [vp, vp]
    L.adascale_set_state.argtypes = [vp, vp]
    L.adascale_step_host.argtypes = [vp, vpp, vpp, vpp, C.POINTER(LrSchedule), C.POINTER(Stats), vp]
    L.adascale_stream_probe.argtypes = [C.c_int32, vp, vp, C.c_int64, vp]
    L.adascale_tiling.argtypes = [C.POINTER(C.c_int64), C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_uint8),
                                  C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.POINTER(C.c_int32),
                                  C.POINTER(C.c_int32)]
    L.adascale_grad_stats_static.argtypes = [vpp, C.c_int32, C.c_int32, C.c_int64, vp, vp, vp]
    L.adascale_launch_count.argtypes = [vp]
    L.adascale_launch_count.restype = C.c_int64
    L.adascale_destroy.argtypes = [vp]
    L.adascale_strerror.argtypes = [C.c_int]
    L.adascale_strerror.restype = C.c_char_p
    L.adascale_last_error.argtypes = [vp]
    L.adascale_last_error.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("adascale_launch_count", "adascale_strerror", "adascale_last_error"):
            getattr(L, name).restype = C.c_int
    return L


lib = _load()


def strerror(status: int) -> str:
    return lib.adascale_strerror(int(status)).decode()


def make_schedule(kind="const", eta0=0.1, d=1.0, T_S1=1.0, milestones=()) -> LrSchedule:
    """Learning-rate families of the paper's App. B.1."""
    s = LrSchedule()
    s.kind = {"const": LR_CONST, "exp": LR_EXP, "step": LR_STEP}[kind]
    s.eta0, s.decay, s.t_s1 = float(eta0), float(d), float(T_S1)
    if len(milestones) > MAX_MILESTONES:
        raise ValueError("at most %d milestones" % MAX_MILESTONES)
    s.n_milestones = len(milestones)
    for i, m in enumerate(milestones):
        s.milestones[i] = float(m)
    return s


def _ptr(x) -> int:
    return x if isinstance(x, int) else x.data_ptr()


def pointer_array(items):
    """ctypes array of addresses from tensors (``data_ptr``) or ints; build once, reuse every step."""
    if isinstance(items, C.Array):
        return items
    flat = []
    for it in items:
        if isinstance(it, (list, tuple)):
            flat.extend(_ptr(x) for x in it)
        else:
            flat.append(_ptr(it))
    return (C.c_void_p * len(flat))(*flat)


def _current_stream(device):
    import torch
    if torch.cuda.is_available():
        return torch.cuda.current_stream(device).cuda_stream
    return 0


class _DeviceSpan:
    """Exposes a raw device range through __cuda_array_interface__ (float32, 1-D)."""

    def __init__(self, ptr, n, owner):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": "<f4", "data": (ptr, False), "version": 3}
        self._owner = owner


class AdaScale:
    """One AdaScale run on one GPU: owns the native context."""

    def __init__(self, numels, S, grad_dtype="f32", momentum=0.0, weight_decay=0.0, eps=1e-6, theta=-1.0,
                 flags=0, device=0, max_S=0):
        self.numels = [int(n) for n in numels]
        self.T = len(self.numels)
        self.S = int(S)
        self.device = int(device)
        self._numel_arr = (C.c_int64 * max(self.T, 1))(*self.numels)
        cfg = Config()
        cfg.S, cfg.max_S, cfg.n_tensors = self.S, int(max_S), self.T
        cfg.grad_dtype = {"f32": F32, "bf16": BF16}.get(grad_dtype, grad_dtype)
        cfg.numel = C.cast(self._numel_arr, C.POINTER(C.c_int64))
        cfg.momentum, cfg.weight_decay, cfg.eps, cfg.theta = momentum, weight_decay, eps, theta
        cfg.flags, cfg.device = int(flags), self.device
        self._ctx = C.c_void_p()
        self._check(lib.adascale_init(C.byref(cfg), C.byref(self._ctx)), init=True)

    # ---- plumbing
    def _check(self, status, init=False):
        if status != OK:
            detail = "" if init or not self._ctx else lib.adascale_last_error(self._ctx).decode()
            raise AdaScaleError(status, strerror(status) + (" (" + detail + ")" if detail else ""))

    def _stream(self, stream):
        return C.c_void_p(_current_stream(self.device) if stream is None else int(stream))

    def close(self):
        if getattr(self, "_ctx", None):
            lib.adascale_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the C ABI, same names
    def step(self, grads, params, momentum, sched, stream=None):
        self._check(lib.adascale_step(self._ctx, pointer_array(grads), pointer_array(params),
                                      pointer_array(momentum), C.byref(sched), self._stream(stream)))

    def reduce(self, grads, sched, stream=None):
        self._check(lib.adascale_reduce(self._ctx, pointer_array(grads), C.byref(sched), self._stream(stream)))

    def update(self, params, momentum, stream=None):
        self._check(lib.adascale_update(self._ctx, pointer_array(params), pointer_array(momentum),
                                        self._stream(stream)))

    def reduce_sums(self, grads, sums, stream=None):
        """Column-sharded use: this shard's mean gradient and its two sums (device float64[2])."""
        self._check(lib.adascale_reduce_sums(self._ctx, pointer_array(grads), C.c_void_p(_ptr(sums)),
                                             self._stream(stream)))

    def apply_sums(self, sums, sched, params, momentum, stream=None):
        """Scalar part on sums completed across shards, then this shard's update."""
        self._check(lib.adascale_apply_sums(self._ctx, C.c_void_p(_ptr(sums)), C.byref(sched),
                                            pointer_array(params), pointer_array(momentum), self._stream(stream)))

    def step_host(self, grads, params, momentum, sched, stream=None) -> Stats:
        out = Stats()
        self._check(lib.adascale_step_host(self._ctx, pointer_array(grads), pointer_array(params),
                                           pointer_array(momentum), C.byref(sched), C.byref(out),
                                           self._stream(stream)))
        return out

    def get_gain_tau(self, blocking=True) -> Stats:
        out = Stats()
        self._check(lib.adascale_get_gain_tau(self._ctx, C.byref(out), 1 if blocking else 0))
        return out

    def mean_grad(self):
        """Device addresses of the float32 mean gradient, one per tensor."""
        arr = (C.c_void_p * self.T)()
        self._check(lib.adascale_mean_grad(self._ctx, arr))
        return [int(p or 0) for p in arr]

    def mean_grad_tensors(self):
        """The mean gradient as torch views of the library's memory (no copy)."""
        import torch
        out = []
        for p, n in zip(self.mean_grad(), self.numels):
            if n == 0:
                out.append(torch.empty(0, dtype=torch.float32, device="cuda:%d" % self.device))
            else:
                out.append(torch.as_tensor(_DeviceSpan(p, n, self), device="cuda:%d" % self.device))
        return out

    def set_scale(self, S):
        self._check(lib.adascale_set_scale(self._ctx, int(S)))
        self.S = int(S)

    def set_wait_limit(self, polls):
        """Bound of the reduce kernel's handshake waits (a test hook for the give-up path)."""
        self._check(lib.adascale_set_wait_limit(self._ctx, int(polls)))

    def set_tile_runs(self, run_tiles):
        """-1: the library chooses; 0: static assignment; n: runs of n tiles from the device counter."""
        self._check(lib.adascale_set_tile_runs(self._ctx, int(run_tiles)))

    def get_state(self) -> bytes:
        buf = C.create_string_buffer(STATE_BYTES)
        self._check(lib.adascale_get_state(self._ctx, buf))
        return buf.raw

    def set_state(self, blob: bytes):
        if len(blob) != STATE_BYTES:
            raise ValueError("state blob must be %d bytes" % STATE_BYTES)
        buf = C.create_string_buffer(blob, STATE_BYTES)
        self._check(lib.adascale_set_state(self._ctx, buf))

    @property
    def launch_count(self) -> int:
        return int(lib.adascale_launch_count(self._ctx))


def tiling(numels, S, grad_dtype="f32", aligned=None, n_blocks=296):
    """Host-only: (staged-tile prefix, scalar-tile prefix, tile columns, rows per stage)."""
    T = len(numels)
    arr = (C.c_int64 * T)(*[int(n) for n in numels])
    al = None if aligned is None else (C.c_uint8 * T)(*[1 if a else 0 for a in aligned])
    tp, sp = (C.c_int64 * (T + 1))(), (C.c_int64 * (T + 1))()
    cols, rows = C.c_int32(), C.c_int32()
    status = lib.adascale_tiling(arr, T, {"f32": F32, "bf16": BF16}.get(grad_dtype, grad_dtype), int(S), al,
                                 int(n_blocks), tp, sp, C.byref(cols), C.byref(rows))
    if status != OK:
        raise AdaScaleError(status, strerror(status))
    return list(tp), list(sp), cols.value, rows.value


STATIC_MAX_ROWS = 32
STATIC_MAX_NUMEL = 2147483640


def grad_stats_static(rows, n, grad_dtype, gbar, sums, stream=None, device=0):
    """Mean gradient and the two sums of one tensor through the entry point that allocates nothing.

    For callers that may not allocate device memory: rows, gbar (float32, n) and sums
    (float64, 2) are the caller's buffers; the library's own scratch is a fixed array.  Calls
    that can overlap on the GPU share that array and must be ordered by the caller.
    """
    s = C.c_void_p(_current_stream(device) if stream is None else int(stream))
    status = lib.adascale_grad_stats_static(pointer_array(rows), len(rows), {"f32": F32, "bf16": BF16}.get(grad_dtype, grad_dtype),
                                            int(n), C.c_void_p(_ptr(gbar)), C.c_void_p(_ptr(sums)), s)
    if status != OK:
        raise AdaScaleError(status, strerror(status))


def stream_probe(kind, a, b, n_bytes, stream=None, device=0):
    """kind 0 read, 1 copy, 2 read-modify-write; a, b tensors or addresses."""
    s = C.c_void_p(_current_stream(device) if stream is None else int(stream))
    status = lib.adascale_stream_probe(int(kind), C.c_void_p(_ptr(a)), C.c_void_p(_ptr(b) if b is not None else 0),
                                       int(n_bytes), s)
    if status != OK:
        raise AdaScaleError(status, strerror(status))
