"""Host-only checks of the C-ABI library: it loads, exports what the header declares and
rejects bad arguments before touching CUDA."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2007_05105_b200 import build
    build.build()
    from paper_2007_05105_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(B):
    header = open(os.path.join(ROOT, "include", "adascale.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(adascale_[a-z_]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    raw = C.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), name


def test_struct_layouts_match_the_header(B):
    assert C.sizeof(B.LrSchedule) == 8 + 3 * 8 + 8 * 8
    assert C.sizeof(B.Stats) == 10 * 8 + 3 * 8 + 8
    assert C.sizeof(B.Config) == 16 + 8 + 4 * 8 + 8
    assert B.STATE_BYTES == 128


def test_strerror(B):
    assert B.strerror(B.OK) == "ok"
    texts = {B.strerror(i) for i in range(6)}
    assert len(texts) == 6
    assert B.strerror(99) == "unknown status"


def _cfg(B, **over):
    numel = (C.c_int64 * 2)(8, 8)
    cfg = B.Config()
    cfg.S, cfg.max_S, cfg.n_tensors, cfg.grad_dtype = 2, 0, 2, B.F32
    cfg.numel = C.cast(numel, C.POINTER(C.c_int64))
    cfg.momentum, cfg.weight_decay, cfg.eps, cfg.theta, cfg.flags, cfg.device = 0.9, 0.0, 1e-6, -1.0, 0, 0
    for k, v in over.items():
        setattr(cfg, k, v)
    cfg._keep = numel
    return cfg


@pytest.mark.parametrize("over", [dict(S=0), dict(n_tensors=0), dict(grad_dtype=7), dict(theta=1.0),
                                  dict(eps=-1.0), dict(max_S=1), dict(flags=64), dict(flags=8), dict(device=-1),
                                  dict(momentum=float("nan"))])
def test_init_rejects_bad_config_without_cuda(B, over):
    ctx = C.c_void_p()
    assert B.lib.adascale_init(C.byref(_cfg(B, **over)), C.byref(ctx)) == B.ERR_INVALID_ARG
    assert not ctx.value


def test_init_rejects_nulls_negative_numel_and_huge_scale(B):
    ctx = C.c_void_p()
    assert B.lib.adascale_init(None, C.byref(ctx)) == B.ERR_INVALID_ARG
    assert B.lib.adascale_init(C.byref(_cfg(B)), None) == B.ERR_INVALID_ARG
    cfg = _cfg(B)
    cfg._keep[1] = -1
    assert B.lib.adascale_init(C.byref(cfg), C.byref(ctx)) == B.ERR_INVALID_ARG
    assert B.lib.adascale_init(C.byref(_cfg(B, S=5000)), C.byref(ctx)) == B.ERR_TOO_LARGE


def test_null_context_is_rejected_everywhere(B):
    sched = B.make_schedule()
    arr = (C.c_void_p * 1)()
    st = B.Stats()
    assert B.lib.adascale_step(None, arr, arr, arr, C.byref(sched), None) == B.ERR_INVALID_ARG
    assert B.lib.adascale_reduce(None, arr, C.byref(sched), None) == B.ERR_INVALID_ARG
    assert B.lib.adascale_update(None, arr, arr, None) == B.ERR_INVALID_ARG
    assert B.lib.adascale_reduce_sums(None, arr, arr, None) == B.ERR_INVALID_ARG
    assert B.lib.adascale_apply_sums(None, arr, C.byref(sched), arr, arr, None) == B.ERR_INVALID_ARG
    assert B.lib.adascale_get_gain_tau(None, C.byref(st), 1) == B.ERR_INVALID_ARG
    assert B.lib.adascale_mean_grad(None, arr) == B.ERR_INVALID_ARG
    assert B.lib.adascale_set_scale(None, 2) == B.ERR_INVALID_ARG
    assert B.lib.adascale_get_state(None, arr) == B.ERR_INVALID_ARG
    assert B.lib.adascale_set_state(None, arr) == B.ERR_INVALID_ARG
    assert B.lib.adascale_step_host(None, arr, arr, arr, C.byref(sched), None, None) == B.ERR_INVALID_ARG
    assert B.lib.adascale_destroy(None) == B.OK
    assert B.lib.adascale_launch_count(None) == 0
    assert B.lib.adascale_last_error(None) == b""
    assert B.lib.adascale_stream_probe(0, None, None, 16, None) == B.ERR_INVALID_ARG
    assert B.lib.adascale_stream_probe(5, 16, 16, 16, None) == B.ERR_INVALID_ARG


def test_without_a_device_init_fails_cleanly(B):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    ctx = C.c_void_p()
    assert B.lib.adascale_init(C.byref(_cfg(B)), C.byref(ctx)) == B.ERR_CUDA
    assert not ctx.value


def test_schedule_builder(B):
    s = B.make_schedule("step", eta0=0.1, d=0.1, milestones=(150240, 300480, 400640))
    assert s.kind == B.LR_STEP and s.n_milestones == 3 and s.milestones[2] == 400640.0
    with pytest.raises(ValueError):
        B.make_schedule("step", milestones=range(9))
