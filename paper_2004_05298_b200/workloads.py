"""Seeded synthetic workloads: shapes, hyper-parameters and gradient streams.

This module only draws random inputs.  It holds none of the method's arithmetic
(no momentum, error feedback, compression, averaging or update), so that the CUDA
library and the CPU oracle can both be fed from it without sharing any of what is
being checked.  Whoever calls it gets torch tensors on the device it names; the
same bits are then handed to both sides.

The paper trains image classifiers (CIFAR-10/100, ImageNet) and prints no model
size; the five workloads below stand in for the flattened gradient streams of
networks of those sizes.  Values never steer control flow in the step, so they
matter for the numerical comparison only.

  1  tiny            d = 1,000,000    W = 4   k = d/32    g ~ N(0, 1e-2) (variance)
  2  resnet56_sized  d =   855,770    W = 8   k = d/32    57 tensors, per-tensor sigma
  3  resnet18_sized  d = 11,689,512   W = 8   k = d/100   1e-3 * Student-t(3), 5 % of entries x10
  4  resnet50_sized  d = 25,557,032   W = 16  k = d/256   161 tensors, per-tensor sigma
  5  vgg16_sized     d = 138,357,544  W = 16  k = d/{8,32,256,1000}   g ~ N(0, 1e-3) (variance)

Unstated hyper-parameters take the paper's experimental values: learning rate 0.1,
momentum 0.9, detach coefficient lambda 0.3.
"""
from dataclasses import dataclass, replace
import math

import numpy as np
import torch

VARIANT_DEF, VARIANT_DEF_A, VARIANT_EF = 0, 1, 2
VARIANT_NAMES = {VARIANT_DEF: "DEF", VARIANT_DEF_A: "DEF-A", VARIANT_EF: "EF"}


@dataclass(frozen=True)
class Workload:
    cfg: int                    # 1..5, also the RBGS seed passed to the step
    name: str
    d: int                      # model size
    W: int                      # workers (the paper's K)
    ratio: int                  # compression ratio d/k
    variant: int
    steps: int
    grad: str                   # "normal" | "per_tensor" | "student_t"
    lr: float = 0.1
    momentum: float = 0.9
    lam: float = 0.3
    sigma: float = 0.0          # "normal": standard deviation
    n_tensors: int = 0          # "per_tensor": how many tensors the flat vector is cut into
    size_range: tuple = (0, 0)  # "per_tensor": tensor sizes are log-uniform in this range
    sigma_range: tuple = (0.0, 0.0)

    @property
    def k(self):
        return max(1, self.d // self.ratio)

    @property
    def rbgs_seed(self):
        return self.cfg

    @property
    def elements_per_step(self):
        return self.W * self.d

    def algorithmic_bytes_per_step(self):
        """Bytes one step has to move: read g, read+write m, read+write e over [W, d]
        (20 B per gradient element; 12 B without momentum) plus read+write of x on the block."""
        per_element = 20 if self.momentum != 0.0 else 12
        return per_element * self.W * self.d + 8 * self.k

    def scaled(self, d, **kw):
        """The same recipe on a smaller model (tests that must finish quickly on a CPU)."""
        lo, hi = self.size_range
        if self.grad == "per_tensor":
            hi = max(lo + 1, min(hi, d // max(1, self.n_tensors // 4)))
        return replace(self, d=int(d), size_range=(lo, hi), **kw)

    def with_ratio(self, ratio, variant=None):
        return replace(self, ratio=int(ratio), variant=self.variant if variant is None else variant)


CONFIGS = {
    1: Workload(1, "tiny", 1_000_000, 4, 32, VARIANT_DEF, 10, "normal", sigma=math.sqrt(1e-2)),
    2: Workload(2, "resnet56_sized", 855_770, 8, 32, VARIANT_DEF_A, 100, "per_tensor",
                n_tensors=57, size_range=(16, 36_864), sigma_range=(1e-4, 1e-1)),
    3: Workload(3, "resnet18_sized", 11_689_512, 8, 100, VARIANT_DEF, 50, "student_t"),
    4: Workload(4, "resnet50_sized", 25_557_032, 16, 256, VARIANT_DEF_A, 20, "per_tensor",
                n_tensors=161, size_range=(64, 2_400_000), sigma_range=(1e-5, 1e-2)),
    5: Workload(5, "vgg16_sized", 138_357_544, 16, 32, VARIANT_DEF, 10, "normal",
                sigma=math.sqrt(1e-3)),
}
CFG5_RATIOS = (8, 32, 256, 1000)
CFG5_VARIANTS = (VARIANT_DEF, VARIANT_EF)


def get(cfg):
    return CONFIGS[int(cfg)]


def tensor_sizes(wl):
    """Sizes of the tensors the flat vector is cut into ("per_tensor" workloads): draw
    log-uniform sizes in size_range, find by bisection the common factor under which the
    clamped, floored sizes sum to d, and give the few coordinates left over to the largest
    tensor.  Seeded by the workload number; same on every device."""
    rng = np.random.default_rng(1000 * wl.cfg + 998)
    lo, hi = wl.size_range
    if not (lo * wl.n_tensors <= wl.d <= hi * wl.n_tensors):
        raise ValueError("cannot cut d = %d into %d tensors within %s" % (wl.d, wl.n_tensors, wl.size_range))
    u = np.exp(rng.uniform(math.log(lo), math.log(hi), size=wl.n_tensors))

    def cut(c):
        return np.clip(np.floor(c * u), lo, hi).astype(np.int64)

    c_lo, c_hi = 0.0, float(hi) / float(u.min()) + 1.0
    for _ in range(200):
        c = 0.5 * (c_lo + c_hi)
        if int(cut(c).sum()) <= wl.d:
            c_lo = c
        else:
            c_hi = c
    sizes = cut(c_lo)
    sizes[int(np.argmax(sizes))] += wl.d - int(sizes.sum())
    assert sizes.min() >= 1 and int(sizes.sum()) == wl.d
    return sizes


def tensor_sigmas(wl):
    rng = np.random.default_rng(1000 * wl.cfg + 997)
    lo, hi = wl.sigma_range
    return np.exp(rng.uniform(math.log(lo), math.log(hi), size=wl.n_tensors)).astype(np.float32)


def column_sigma(wl, device):
    """[d] float32: the gradient standard deviation of each coordinate ("per_tensor")."""
    sizes = torch.from_numpy(tensor_sizes(wl)).to(device)
    sigmas = torch.from_numpy(tensor_sigmas(wl)).to(device)
    return torch.repeat_interleave(sigmas, sizes)


def _generator(device, seed):
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    return gen


def initial_params(wl, device):
    """x_0 = y_0 ~ N(0, 0.05^2) (the paper only says x_0 = y_0)."""
    gen = _generator(device, 1000 * wl.cfg + 999)
    return torch.empty(wl.d, dtype=torch.float32, device=device).normal_(0.0, 0.05, generator=gen)


def zeros_state(wl, device):
    """e_{k,0} = 0 and m_{k,0} = 0 as [W, d] tensors."""
    e = torch.zeros(wl.W, wl.d, dtype=torch.float32, device=device)
    m = torch.zeros(wl.W, wl.d, dtype=torch.float32, device=device)
    return e, m


def gradients(wl, step, device, out=None, col_sigma=None):
    """The [W, d] gradients of one step, seeded by (workload, step)."""
    gen = _generator(device, 1000 * wl.cfg + int(step))
    g = out if out is not None else torch.empty(wl.W, wl.d, dtype=torch.float32, device=device)
    if wl.grad == "normal":
        g.normal_(0.0, wl.sigma, generator=gen)
    elif wl.grad == "per_tensor":
        if col_sigma is None:
            col_sigma = column_sigma(wl, device)
        g.normal_(0.0, 1.0, generator=gen)
        g.mul_(col_sigma.unsqueeze(0))
    elif wl.grad == "student_t":
        # t_3 = Z / sqrt(chi2_3 / 3), one row at a time to bound the temporaries
        for w in range(wl.W):
            z = torch.empty(4, wl.d, dtype=torch.float32, device=device).normal_(generator=gen)
            chi2 = (z[1:] * z[1:]).sum(dim=0)
            row = z[0] * torch.rsqrt(chi2 / 3.0) * 1e-3
            big = torch.empty(wl.d, dtype=torch.float32, device=device).uniform_(generator=gen) < 0.05
            g[w] = torch.where(big, row * 10.0, row)
    else:
        raise ValueError(wl.grad)
    return g


def shard_columns(d, world_size, rank, align=4):
    """Contiguous column range [j0, j1) of rank `rank` when d coordinates are cut across
    world_size ranks; boundaries are multiples of `align` so every shard keeps 16-byte rows."""
    per = -(-d // world_size)
    per = -(-per // align) * align
    j0 = min(d, rank * per)
    j1 = min(d, j0 + per)
    return j0, j1
