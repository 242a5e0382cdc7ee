"""Seeded synthetic workloads: segment tables and value generators.

This module holds no arithmetic of the optimizer pass itself.  It only lays out
parameter tensors of public architectures in a flat buffer and draws seeded random
values with the distributions the five benchmark configurations prescribe.  Both the
CUDA library's callers and the CPU checker's callers take their inputs from here.

Values stand in for real training tensors (CIFAR / ImageNet models, a GPT-style
decoder): shapes are the architectures' parameter shapes, values are synthetic.
"""
from dataclasses import dataclass, field
import math

import torch

ALIGN = 8  # segment offsets are padded up to a multiple of this many elements


def _prod(shape):
    n = 1
    for s in shape:
        n *= s
    return n


def mlp_tiny_shapes():
    return [(256, 784), (256,), (10, 256), (10,)]


def resnet18_cifar_shapes(num_classes=10, width=64):
    s = [(width, 3, 3, 3), (width,), (width,)]
    inp = width
    for stage, planes in enumerate([width, 2 * width, 4 * width, 8 * width]):
        for block in range(2):
            s += [(planes, inp, 3, 3), (planes,), (planes,), (planes, planes, 3, 3), (planes,), (planes,)]
            if block == 0 and stage > 0:
                s += [(planes, inp, 1, 1), (planes,), (planes,)]
            inp = planes
    s += [(num_classes, inp), (num_classes,)]
    return s


def efficientnet_b0_shapes(num_classes=10):
    s = [(32, 3, 3, 3), (32,), (32,)]
    expand = [1, 6, 6, 6, 6, 6, 6]
    kernel = [3, 3, 5, 3, 5, 5, 3]
    out_ch = [16, 24, 40, 80, 112, 192, 320]
    repeats = [1, 2, 2, 3, 3, 4, 1]
    inp = 32
    for e, k, o, r in zip(expand, kernel, out_ch, repeats):
        for _ in range(r):
            mid = inp * e
            if e != 1:
                s += [(mid, inp, 1, 1), (mid,), (mid,)]
            s += [(mid, 1, k, k), (mid,), (mid,)]
            sq = max(1, inp // 4)
            s += [(sq, mid, 1, 1), (sq,), (mid, sq, 1, 1), (mid,)]
            s += [(o, mid, 1, 1), (o,), (o,)]
            inp = o
    s += [(1280, inp, 1, 1), (1280,), (1280,)]
    s += [(num_classes, 1280), (num_classes,)]
    return s


def resnet50_shapes(num_classes=1000, width=64):
    s = [(width, 3, 7, 7), (width,), (width,)]
    inp = width
    for planes, blocks in zip([width, 2 * width, 4 * width, 8 * width], [3, 4, 6, 3]):
        for block in range(blocks):
            s += [(planes, inp, 1, 1), (planes,), (planes,), (planes, planes, 3, 3), (planes,), (planes,),
                  (4 * planes, planes, 1, 1), (4 * planes,), (4 * planes,)]
            if block == 0:
                s += [(4 * planes, inp, 1, 1), (4 * planes,), (4 * planes,)]
            inp = 4 * planes
    s += [(num_classes, inp), (num_classes,)]
    return s


def gpt_shapes(layers=24, d=2048, vocab=50304):
    s = [(vocab, d)]
    for _ in range(layers):
        s += [(d,), (3 * d, d), (d, d), (d,), (4 * d, d), (d, 4 * d)]
    return s


def segment_table(shapes, align=ALIGN):
    """[(offset, length)] in elements, offsets padded up to `align`; returns (table, n_total)."""
    table, off = [], 0
    for sh in shapes:
        n = _prod(sh)
        if align > 1:
            off = (off + align - 1) // align * align
        table.append((off, n))
        off += n
    n_total = (off + 7) // 8 * 8
    return table, n_total


@dataclass
class Workload:
    name: str
    shapes: list
    steps: int
    grad_dtype: str = "f32"
    num_probes: int = 1
    topk_ppm: int = 1000000
    tau_low: float = 1e-7
    tau_high: float = 1e-5
    tau_curv: float = 0.9
    beta: float = 0.9
    alpha: float = 1.0
    eta0: float = 0.1
    t_ctrl: int = 1
    d_low: float = 1e-5
    d_high: float = 1.0
    grad_recipe: str = "layer_loguniform"   # "pow2_per_layer" | "layer_loguniform" | "heavy_tail"
    seed: int = 1234
    probe_seed: int = 0
    align: int = ALIGN
    table: list = field(default_factory=list)
    n_total: int = 0

    def __post_init__(self):
        self.table, self.n_total = segment_table(self.shapes, self.align)

    @property
    def num_params(self):
        return sum(n for _, n in self.table)

    def hparams(self):
        return dict(beta=self.beta, tau_low=self.tau_low, tau_high=self.tau_high, tau_curv=self.tau_curv,
                    alpha=self.alpha, eta0=self.eta0, topk_ppm=self.topk_ppm, num_probes=self.num_probes,
                    t_ctrl=self.t_ctrl, grad_dtype=self.grad_dtype)


def get(name, **overrides):
    """The five benchmark configurations (and scaled-down variants through overrides)."""
    if name == "mlp_tiny":
        w = dict(shapes=mlp_tiny_shapes(), steps=10, tau_low=2e-6, tau_high=2e-5, d_low=1e-4,
                 grad_recipe="pow2_per_layer")
    elif name == "resnet18_cifar":
        w = dict(shapes=resnet18_cifar_shapes(), steps=100)
    elif name == "efficientnet_b0_cifar":
        w = dict(shapes=efficientnet_b0_shapes(), steps=100)
    elif name == "resnet50_topk":
        w = dict(shapes=resnet50_shapes(), steps=50, num_probes=4, topk_ppm=100000, grad_recipe="heavy_tail")
    elif name == "gpt_1p3b":
        w = dict(shapes=gpt_shapes(), steps=20, grad_dtype="bf16", d_low=1e-6)
    elif name == "gpt_1block":
        # one decoder block plus the embedding: the 1.3B workload's tensor mix at a size a profiler can replay
        w = dict(shapes=gpt_shapes(layers=1), steps=20, grad_dtype="bf16", d_low=1e-6)
    elif name == "gpt_3block":
        # three decoder blocks behind a small embedding: layers of the 1.3B workload's sizes, no tensor beyond L2
        w = dict(shapes=gpt_shapes(layers=3, vocab=8192), steps=20, grad_dtype="bf16", d_low=1e-6)
    else:
        raise KeyError(name)
    w.update(overrides)
    return Workload(name=name, **w)


NAMES = ["mlp_tiny", "resnet18_cifar", "efficientnet_b0_cifar", "resnet50_topk", "gpt_1p3b"]


def _gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    return g


def _mix(seed, salt, t=0):
    return (seed * 1000003 + salt * 7919 + t * 104729 + 12345) % (2 ** 62)


def layer_scales(wl: Workload):
    """Per-layer gradient standard deviations (host list of floats)."""
    L = len(wl.table)
    if wl.grad_recipe == "pow2_per_layer":
        return [1e-3 * 2.0 ** l for l in range(L)]
    if wl.grad_recipe == "heavy_tail":
        return [1e-3] * L
    u = torch.rand(L, generator=_gen(_mix(wl.seed, 1), "cpu"), dtype=torch.float64)
    return [1e-3 * 0.1 * math.exp(float(x) * math.log(100.0)) for x in u]


def make_weights(wl: Workload, device="cpu"):
    """w ~ N(0, 0.05) over the whole flat buffer (gaps included; the pass never touches gaps)."""
    return torch.randn(wl.n_total, generator=_gen(_mix(wl.seed, 2), device), device=device,
                       dtype=torch.float32) * 0.05


def make_curvature(wl: Workload, device="cpu"):
    """D ~ LogUniform[d_low, d_high] per element, float32."""
    u = torch.rand(wl.n_total, generator=_gen(_mix(wl.seed, 3), device), device=device, dtype=torch.float32)
    return wl.d_low * torch.exp(u * math.log(wl.d_high / wl.d_low))


def make_grads(wl: Workload, t: int, device="cpu"):
    """Gradient of step t: float32 [n_total], or bfloat16 when the workload says so."""
    gen = _gen(_mix(wl.seed, 4, t), device)
    g = torch.randn(wl.n_total, generator=gen, device=device, dtype=torch.float32)
    for (off, n), s in zip(wl.table, layer_scales(wl)):
        g[off:off + n] *= s
    if wl.grad_recipe == "heavy_tail":
        # 1 % of the elements: 1e-3 * Student-t(nu=2) = N(0,1) / sqrt(Exp(1))
        pick = torch.rand(wl.n_total, generator=gen, device=device) < 0.01
        zn = torch.randn(wl.n_total, generator=gen, device=device, dtype=torch.float32)
        ex = -torch.log1p(-torch.rand(wl.n_total, generator=gen, device=device, dtype=torch.float32))
        heavy = 1e-3 * zn / torch.sqrt(ex.clamp_min(1e-12))
        g = torch.where(pick, heavy, g)
    if wl.grad_dtype == "bf16":
        g = g.to(torch.bfloat16)
    return g
