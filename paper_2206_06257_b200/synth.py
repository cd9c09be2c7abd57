"""Seeded synthetic inputs: parameter-tensor shape lists and value generators.

This module holds NONE of the method's arithmetic (no quantizer, no aggregation,
no update rule, no random-number scheme of the method).  It only produces the
inputs -- layer sizes, parameters, momentum and the M workers' gradient buffers --
that both the CUDA path and the CPU checker consume, so that the two can be run
on identical data.

The shapes are those of the networks the paper trains (ResNet-18 on CIFAR-10,
ResNet-50 on ImageNet; Sec. 6 "Experiment setup"); the values are synthetic
stand-ins for adversarial-minibatch gradients, drawn from explicitly seeded
torch generators.  Nothing here reads a dataset or a checkpoint.
"""
from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np
import torch


# ----------------------------------------------------------------------------
# Shape lists.  One entry per parameter tensor: (name, numel, kind, fan_in).
# kind in {"weight", "bn_weight", "bias"}.
# ----------------------------------------------------------------------------

def _conv(name, cout, cin, k):
    return (name, cout * cin * k * k, "weight", cin * k * k)


def _bn(name, c):
    return [(name + ".weight", c, "bn_weight", 0), (name + ".bias", c, "bias", 0)]


def tiny_mlp_tensors():
    """784-256-128-10 perceptron: 6 tensors, 235,146 parameters."""
    t = []
    for k, (fin, fout) in enumerate([(784, 256), (256, 128), (128, 10)]):
        t.append(("fc%d.weight" % k, fin * fout, "weight", fin))
        t.append(("fc%d.bias" % k, fout, "bias", 0))
    return t


def resnet18_cifar_tensors(num_classes=10):
    """ResNet-18 with the CIFAR stem (3x3 conv, no max-pool): 62 tensors, 11,173,962 parameters."""
    t = [_conv("conv1", 64, 3, 3)] + _bn("bn1", 64)
    cin = 64
    for s, w in enumerate([64, 128, 256, 512]):
        for b in range(2):
            p = "layer%d.%d" % (s + 1, b)
            t.append(_conv(p + ".conv1", w, cin, 3)); t += _bn(p + ".bn1", w)
            t.append(_conv(p + ".conv2", w, w, 3)); t += _bn(p + ".bn2", w)
            if b == 0 and cin != w:
                t.append(_conv(p + ".downsample.0", w, cin, 1)); t += _bn(p + ".downsample.1", w)
            cin = w
    t.append(("fc.weight", num_classes * 512, "weight", 512))
    t.append(("fc.bias", num_classes, "bias", 0))
    return t


def resnet50_tensors(num_classes=1000):
    """ResNet-50 (bottleneck, [3,4,6,3]): 161 tensors, 25,557,032 parameters."""
    t = [_conv("conv1", 64, 3, 7)] + _bn("bn1", 64)
    cin = 64
    for s, (w, nblk) in enumerate(zip([64, 128, 256, 512], [3, 4, 6, 3])):
        for b in range(nblk):
            p = "layer%d.%d" % (s + 1, b)
            t.append(_conv(p + ".conv1", w, cin, 1)); t += _bn(p + ".bn1", w)
            t.append(_conv(p + ".conv2", w, w, 3)); t += _bn(p + ".bn2", w)
            t.append(_conv(p + ".conv3", 4 * w, w, 1)); t += _bn(p + ".bn3", 4 * w)
            if b == 0:
                t.append(_conv(p + ".downsample.0", 4 * w, cin, 1)); t += _bn(p + ".downsample.1", 4 * w)
            cin = 4 * w
    t.append(("fc.weight", num_classes * 2048, "weight", 2048))
    t.append(("fc.bias", num_classes, "bias", 0))
    return t


def flat_tensors(total=1_000_000_000, num_layers=400, lo=64, hi=16 * 1024 * 1024, seed=0):
    """num_layers sizes, log-uniform on [lo, hi], rescaled so that they sum to `total`
    (clipped to [lo, hi]; the remainder goes to the largest tensor).  Sizes are NOT
    forced to multiples of 4."""
    rng = np.random.RandomState(seed)
    raw = np.exp(rng.uniform(np.log(lo), np.log(hi), size=num_layers))
    sizes = raw.copy()
    for _ in range(64):                       # rescale/clip until the clipped sum is close
        free = (sizes > lo) & (sizes < hi)
        fixed = sizes[~free].sum()
        if not free.any():
            break
        sizes[free] *= (total - fixed) / sizes[free].sum()
        sizes = np.clip(sizes, lo, hi)
        if abs(sizes.sum() - total) < 1:
            break
    sizes = np.floor(sizes).astype(np.int64)
    sizes = np.clip(sizes, lo, hi)
    k = int(np.argmax(sizes))
    sizes[k] += total - int(sizes.sum())
    assert sizes.sum() == total and sizes.min() >= 1
    return [("flat%d" % i, int(n), "weight", 1024) for i, n in enumerate(sizes)]


# ----------------------------------------------------------------------------
# Workload configurations.
# ----------------------------------------------------------------------------

@dataclass
class Config:
    name: str
    tensors: List[Tuple[str, int, str, int]]
    M: int
    bits: int
    lr: float = 0.1
    momentum: float = 0.9
    weight_decay: float = 5e-4
    c_l: float = 0.0
    c_u: float = 10.0
    steps: int = 1
    grad_dist: str = "normal"               # "normal" | "student_t3"
    log10_sigma: Tuple[float, float] = (-4.0, -1.0)
    theta_init: str = "kaiming"             # "kaiming" | "normal:<std>"
    mom_std: float = 0.0
    zero_grad_layers: Tuple[int, ...] = ()
    zero_param_layers: Tuple[int, ...] = ()
    seed: int = 0
    rng_bits: int = 16                      # resolution of the quantizer's uniform number (16 or 23)
    offsets: np.ndarray = field(init=False)

    def __post_init__(self):
        sizes = np.array([t[1] for t in self.tensors], dtype=np.int64)
        self.offsets = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)

    @property
    def d(self):
        return int(self.offsets[-1])

    @property
    def h(self):
        return len(self.tensors)


def config(name: str, **over) -> Config:
    """The five workloads: 'tiny_mlp', 'resnet18', 'resnet50', 'resnet50_m32', 'flat1b'
    (plus 'flat_small', a scaled-down flat model with odd sizes, for tests)."""
    if name == "tiny_mlp":
        c = Config(name, tiny_mlp_tensors(), M=4, bits=8, lr=0.1, momentum=0.9, weight_decay=5e-4,
                   log10_sigma=(-4.0, -1.0), theta_init="normal:0.05", mom_std=0.0)
    elif name == "resnet18":
        c = Config(name, resnet18_cifar_tensors(), M=6, bits=8, steps=10, log10_sigma=(-4.0, -1.0))
    elif name == "resnet50":
        c = Config(name, resnet50_tensors(), M=8, bits=8, log10_sigma=(-5.0, -1.0), mom_std=1e-3)
    elif name == "resnet50_m32":
        c = Config(name, resnet50_tensors(), M=32, bits=4, log10_sigma=(-5.0, -1.0), mom_std=1e-3,
                   grad_dist="student_t3", zero_grad_layers=(57,), zero_param_layers=(99,))
    elif name == "flat1b":
        c = Config(name, flat_tensors(), M=8, bits=8, log10_sigma=(-5.0, -1.0),
                   theta_init="normal:0.02", mom_std=1e-3)
    elif name == "flat_small":
        c = Config(name, flat_tensors(total=3_000_017, num_layers=40, lo=5, hi=700_001, seed=1), M=3, bits=4,
                   log10_sigma=(-5.0, -1.0), theta_init="normal:0.02", mom_std=1e-3)
    else:
        raise KeyError(name)
    for k, v in over.items():
        setattr(c, k, v)
    return c


# ----------------------------------------------------------------------------
# Value generators (torch; any device).  Every stream has its own derived seed.
# ----------------------------------------------------------------------------

def _gen(device, *key):
    g = torch.Generator(device=device)
    s = 0x9E3779B97F4A7C15
    for k in key:
        s = (s * 6364136223846793005 + 1442695040888963407 + int(k)) % (1 << 63)
    g.manual_seed(s)
    return g


def layer_sigmas(cfg: Config) -> np.ndarray:
    """Per-layer gradient scale sigma_l, log-uniform; the same for every worker and step."""
    rng = np.random.RandomState(cfg.seed + 12345)
    lo, hi = cfg.log10_sigma
    return (10.0 ** rng.uniform(lo, hi, size=cfg.h)).astype(np.float32)


def _per_element(cfg: Config, per_layer: np.ndarray, device) -> torch.Tensor:
    sizes = torch.from_numpy(np.diff(cfg.offsets))
    v = torch.from_numpy(np.asarray(per_layer, dtype=np.float32))
    return torch.repeat_interleave(v, sizes).to(device)


def make_params(cfg: Config, device="cpu"):
    """(theta, mom): float32 [d] each."""
    d = cfg.d
    g = _gen(device, cfg.seed, 1)
    z = torch.randn(d, generator=g, device=device, dtype=torch.float32)
    if cfg.theta_init.startswith("normal:"):
        theta = z * float(cfg.theta_init.split(":")[1])
    else:
        std = np.zeros(cfg.h, dtype=np.float32)
        shift = np.zeros(cfg.h, dtype=np.float32)
        for l, (_, _, kind, fan_in) in enumerate(cfg.tensors):
            if kind == "weight":
                std[l] = np.sqrt(2.0 / fan_in)
            elif kind == "bn_weight":
                std[l], shift[l] = 0.0, 1.0
            else:
                std[l] = 0.01
        theta = z * _per_element(cfg, std, device) + _per_element(cfg, shift, device)
    if cfg.mom_std > 0:
        gm = _gen(device, cfg.seed, 2)
        mom = torch.randn(d, generator=gm, device=device, dtype=torch.float32) * cfg.mom_std
    else:
        mom = torch.zeros(d, device=device, dtype=torch.float32)
    for l in cfg.zero_param_layers:
        theta[int(cfg.offsets[l]):int(cfg.offsets[l + 1])] = 0.0
    return theta.contiguous(), mom.contiguous()


def make_grads(cfg: Config, step: int = 0, device="cpu", sigma_elem=None):
    """List of M float32 [d] gradient buffers for the given step."""
    if sigma_elem is None:
        sigma_elem = _per_element(cfg, layer_sigmas(cfg), device)
    out = []
    for i in range(cfg.M):
        g = _gen(device, cfg.seed, 3, step, i)
        z = torch.randn(cfg.d, generator=g, device=device, dtype=torch.float32)
        if cfg.grad_dist == "student_t3":
            chi = torch.zeros(cfg.d, device=device, dtype=torch.float32)
            for _ in range(3):
                w = torch.randn(cfg.d, generator=g, device=device, dtype=torch.float32)
                chi += w * w
            z = z / torch.sqrt(chi / 3.0)
            del chi, w
        z *= sigma_elem
        for l in cfg.zero_grad_layers:
            z[int(cfg.offsets[l]):int(cfg.offsets[l + 1])] = 0.0
        out.append(z.contiguous())
    return out
