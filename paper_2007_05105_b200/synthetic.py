"""Seeded synthetic gradients with the shapes of the paper's benchmarks.

The paper trains ResNet-18/50, a Transformer and others on public datasets
(Table 1); none of that is available offline, so the gradients here are random
stand-ins with the same tensor lists: g_i = m + s * n_i, a mean m shared by the
S rows plus independent unit-variance noise n_i.  The ratio k = s / std(m)
sets where the gain ratio of Eq. 3 lands between 1 and S.

This module only draws numbers and lays out tensors.  It contains none of the
method's arithmetic and is the one piece that both the CUDA tests/benchmark and
the CPU oracle's callers may share.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch

# --------------------------------------------------------------------------
# tensor lists, generated from architecture hyper-parameters
# --------------------------------------------------------------------------


def _conv(cin, cout, k):
    return (cout, cin, k, k)


def _norm(c):
    return [(c,), (c,)]


def resnet18_shapes(width=64, classes=1000):
    """Basic-block residual network: 7x7 stem, 4 stages of 2 blocks, linear head."""
    shapes = [_conv(3, width, 7)] + _norm(width)
    cin = width
    for stage in range(4):
        cout = width << stage
        for block in range(2):
            shapes += [_conv(cin, cout, 3)] + _norm(cout) + [_conv(cout, cout, 3)] + _norm(cout)
            if block == 0 and stage > 0:
                shapes += [_conv(cin, cout, 1)] + _norm(cout)
            cin = cout
    return shapes + [(classes, cin), (classes,)]


def resnet50_shapes(width=64, classes=1000):
    """Bottleneck residual network: 1x1 / 3x3 / 1x1 blocks (expansion 4), counts 3/4/6/3."""
    shapes = [_conv(3, width, 7)] + _norm(width)
    cin = width
    for stage, blocks in enumerate((3, 4, 6, 3)):
        mid = width << stage
        cout = 4 * mid
        for block in range(blocks):
            shapes += [_conv(cin, mid, 1)] + _norm(mid) + [_conv(mid, mid, 3)] + _norm(mid)
            shapes += [_conv(mid, cout, 1)] + _norm(cout)
            if block == 0:
                shapes += [_conv(cin, cout, 1)] + _norm(cout)
            cin = cout
    return shapes + [(classes, cin), (classes,)]


def _linear(din, dout):
    return [(dout, din), (dout,)]


def transformer_base_shapes(d=512, ffn=2048, layers=6, vocab=32768):
    """Encoder-decoder Transformer with one shared embedding table."""
    shapes = [(vocab, d)]
    for _ in range(layers):  # encoder: self-attention (q, k, v, o), feed-forward, 2 layer norms
        for _ in range(4):
            shapes += _linear(d, d)
        shapes += _linear(d, ffn) + _linear(ffn, d) + _norm(d) + _norm(d)
    for _ in range(layers):  # decoder: self- and cross-attention, feed-forward, 3 layer norms
        for _ in range(8):
            shapes += _linear(d, d)
        shapes += _linear(d, ffn) + _linear(ffn, d) + _norm(d) + _norm(d) + _norm(d)
    return shapes + _norm(d) + _norm(d)


def decoder_24l_shapes(d=1024, ffn=4096, layers=24, vocab=50257, positions=1024):
    """Decoder-only Transformer: token and position tables, fused QKV, pre-norm blocks."""
    shapes = [(vocab, d), (positions, d)]
    for _ in range(layers):
        shapes += _norm(d) + _linear(d, 3 * d) + _linear(d, d) + _norm(d) + _linear(d, ffn) + _linear(ffn, d)
    return shapes + _norm(d)


def numel(shape):
    return int(math.prod(shape))


# --------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------


@dataclass
class Workload:
    name: str
    shapes: list
    S: int
    grad_dtype: str = "f32"          # "f32" | "bf16"
    k: tuple = (1.0, 1.0)            # s / std(m) at the first and the last step (linear in between)
    noise: str = "normal"            # "normal" | "student3" (Student-t, 3 d.o.f., unit variance)
    mean_std: float = 0.1
    momentum: float = 0.9
    weight_decay: float = 0.0
    lr: dict = field(default_factory=lambda: {"kind": "const", "eta0": 0.1})
    steps: int = 10
    seed: int = 2007051050

    @property
    def numels(self):
        return [numel(s) for s in self.shapes]

    @property
    def P(self):
        return sum(self.numels)

    def k_at(self, step):
        if self.steps <= 1:
            return self.k[0]
        return self.k[0] + (self.k[1] - self.k[0]) * step / (self.steps - 1)


def workload(name: str, **over) -> Workload:
    """The five benchmark configurations (and reduced-width variants for the tests)."""
    if name == "single_1m":
        w = Workload(name, [(1 << 20,)], S=4, k=(10.0, 10.0), steps=10, seed=2007051051)
    elif name == "resnet18":
        w = Workload(name, resnet18_shapes(), S=8, k=(3.0, 3.0), weight_decay=1e-4, steps=20,
                     lr={"kind": "step", "eta0": 0.1, "d": 0.1, "milestones": (20.0, 40.0)}, seed=2007051052)
    elif name == "resnet50":
        w = Workload(name, resnet50_shapes(), S=16, grad_dtype="bf16", k=(3.0, 3.0), weight_decay=1e-4,
                     steps=1000, lr={"kind": "step", "eta0": 0.1, "d": 0.1, "milestones": (2000.0, 4000.0)},
                     seed=2007051053)
    elif name == "transformer_base":
        w = Workload(name, transformer_base_shapes(), S=32, k=(3.0, 3.0), noise="student3", momentum=0.99,
                     steps=20, lr={"kind": "step", "eta0": 0.01, "d": 0.1, "milestones": (200.0,)},
                     seed=2007051054)
    elif name == "decoder_24l":
        w = Workload(name, decoder_24l_shapes(), S=32, grad_dtype="bf16", k=(0.1, 10.0), steps=200,
                     lr={"kind": "exp", "eta0": 0.1, "d": 0.05, "T_S1": 5000.0}, seed=2007051055)
    elif name == "decoder_4l":
        # decoder_24l cut to 4 layers and a 16k vocabulary (68M parameters, 4.4 GB of gradients): small
        # enough for a profiler capture, large enough to take the same kernel paths as decoder_24l
        w = Workload(name, decoder_24l_shapes(layers=4, vocab=16384), S=32, grad_dtype="bf16", k=(0.1, 10.0), steps=200,
                     lr={"kind": "exp", "eta0": 0.1, "d": 0.05, "T_S1": 5000.0}, seed=2007051056)
    else:
        raise KeyError(name)
    for key, val in over.items():
        setattr(w, key, val)
    return w


WORKLOAD_NAMES = ("single_1m", "resnet18", "resnet50", "transformer_base", "decoder_24l")


# --------------------------------------------------------------------------
# gradient source
# --------------------------------------------------------------------------


def _torch_dtype(name):
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


class GradientSource:
    """Owns S flat gradient rows and refills them, seeded, for a given step.

    Every row is one flat buffer; tensor k of row i is a view at an offset
    rounded up to ``align`` elements, so pointers stay fixed across steps.
    """

    def __init__(self, wl: Workload, device="cpu", align=64):
        self.wl = wl
        self.device = torch.device(device)
        self.numels = wl.numels
        self.offsets = []
        off = 0
        for n in self.numels:
            self.offsets.append(off)
            off += -(-n // align) * align
        self.flat_len = off
        dt = _torch_dtype(wl.grad_dtype)
        self.gen = torch.Generator(device=self.device)
        self.gen.manual_seed(wl.seed)
        self.mean = torch.empty(self.flat_len, dtype=torch.float32, device=self.device)
        self.mean.normal_(0.0, wl.mean_std, generator=self.gen)
        self.rows = [torch.zeros(self.flat_len, dtype=dt, device=self.device) for _ in range(wl.S)]
        self._tmp = None

    def views(self, flat):
        return [flat[o:o + n] for o, n in zip(self.offsets, self.numels)]

    def _noise(self, out, chunk):
        if self.wl.noise == "normal":
            out.normal_(0.0, 1.0, generator=self.gen)
        elif self.wl.noise == "student3":
            # z / sqrt(chi2_3) is Student-t with 3 degrees of freedom divided by sqrt(3): unit variance
            out.normal_(0.0, 1.0, generator=self.gen)
            den = torch.zeros_like(out)
            for _ in range(3):
                chunk.normal_(0.0, 1.0, generator=self.gen)
                den.addcmul_(chunk, chunk)
            out.div_(den.sqrt_())
        else:
            raise KeyError(self.wl.noise)

    def fill(self, step: int, k: float | None = None):
        """Refill all rows for iteration ``step``; returns grads[i][k] views."""
        wl = self.wl
        s = (wl.k_at(step) if k is None else k) * wl.mean_std
        block = min(self.flat_len, 1 << 26)
        if self._tmp is None:
            self._tmp = (torch.empty(block, dtype=torch.float32, device=self.device),
                         torch.empty(block, dtype=torch.float32, device=self.device))
        for i, row in enumerate(self.rows):
            self.gen.manual_seed(wl.seed + 1000003 * (step + 1) + 7919 * (i + 1))
            for lo in range(0, self.flat_len, block):
                hi = min(lo + block, self.flat_len)
                noise, aux = self._tmp[0][:hi - lo], self._tmp[1][:hi - lo]
                if s == 0.0:
                    noise.zero_()
                else:
                    self._noise(noise, aux)
                noise.mul_(s).add_(self.mean[lo:hi])
                row[lo:hi].copy_(noise)  # rounds to nearest even when the row is bf16
        return self.grads()

    def grads(self):
        return [self.views(r) for r in self.rows]

    def init_params(self, std=1.0):
        """Seeded fp32 parameters and zero momentum with the same layout."""
        self.gen.manual_seed(self.wl.seed + 17)
        w = torch.empty(self.flat_len, dtype=torch.float32, device=self.device)
        w.normal_(0.0, std, generator=self.gen)
        v = torch.zeros(self.flat_len, dtype=torch.float32, device=self.device)
        return w, v
