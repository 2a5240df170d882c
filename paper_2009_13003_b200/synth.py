"""Seeded synthetic model states and deltas.

Only random-number recipes live here: shapes, sizes and value distributions of the workloads. None of
the method's arithmetic (no bucketing, no coding) is in this module, so both the CUDA library's tests
and the CPU oracle's tests can draw their inputs from it. A tensor is generated once, on one device,
and the same bytes are handed to whoever needs them (transcendental functions differ between CPU and
GPU, so nothing may depend on regenerating an input elsewhere).

Stand-ins: the paper evaluates on deltas from training MLR / LeNet-5 / AlexNet / MF on MNIST,
FashionMNIST, Jester and MovieLens. Those are not available; these recipes only take the sizes of
well-known model states and plausible update distributions.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch

SEED0 = 2009130030
_SLICE = 1 << 26  # elements generated at a time, bounds temporary memory


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _fill(n, device, seed, draw):
    """out[i] for i in [0, n), produced slice by slice with one generator."""
    g = _gen(device, seed)
    out = torch.empty(n, dtype=torch.float32, device=device)
    for lo in range(0, n, _SLICE):
        hi = min(n, lo + _SLICE)
        out[lo:hi] = draw(hi - lo, g)
    return out


def normal(n, std, device, seed):
    return _fill(n, device, seed, lambda m, g: torch.randn(m, generator=g, device=device) * std)


def laplace(n, scale, device, seed):
    def draw(m, g):
        u = torch.rand(m, generator=g, device=device) - 0.5
        # rand() can return exactly 0, i.e. |u| = 0.5 and an infinite draw: keep |u| below one half
        return -scale * torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp_(max=0.5 - 2.0 ** -25))

    return _fill(n, device, seed, draw)


def student_t3(n, scale, device, seed):
    def draw(m, g):
        z = torch.randn(m, generator=g, device=device)
        c = torch.randn(3, m, generator=g, device=device).square_().sum(0)
        return scale * z / torch.sqrt(c / 3.0)

    return _fill(n, device, seed, draw)


def lognormal_signed(n, median, sigma, device, seed):
    def draw(m, g):
        mag = torch.exp(torch.randn(m, generator=g, device=device) * sigma + math.log(median))
        sgn = torch.randint(0, 2, (m,), generator=g, device=device, dtype=torch.int8)
        return torch.where(sgn.bool(), mag, -mag)

    return _fill(n, device, seed, draw)


def one_exponent(n, lo_pow, device, seed, two_sign):
    """|d| uniform in [2^lo_pow, 2^(lo_pow+1)): every element falls into one exponent bucket."""

    def draw(m, g):
        mag = (1.0 + torch.rand(m, generator=g, device=device)) * (2.0 ** lo_pow)
        top = torch.tensor(2.0 ** (lo_pow + 1), dtype=torch.float32)
        mag = torch.clamp(mag, max=float(torch.nextafter(top, torch.tensor(0.0))))  # largest fp32 below 2^(lo_pow+1)
        if not two_sign:
            return mag
        sgn = torch.randint(0, 2, (m,), generator=g, device=device, dtype=torch.int8)
        return torch.where(sgn.bool(), mag, -mag)

    return _fill(n, device, seed, draw)


# Parameter-tensor sizes of a ResNet-18-shaped state (conv / batch-norm / fc tensors, sizes only).
def resnet18_segments():
    seg = [64 * 3 * 7 * 7, 64, 64]
    cin = 64
    for cout in (64, 128, 256, 512):
        for block in range(2):
            first_in = cin if block == 0 else cout
            seg += [cout * first_in * 9, cout, cout, cout * cout * 9, cout, cout]
            if block == 0 and cin != cout:
                seg += [cout * cin, cout, cout]
        cin = cout
    seg += [1000 * 512, 1000]
    assert len(seg) == 62 and sum(seg) == 11_689_512
    return seg


@dataclass(frozen=True)
class Config:
    name: str
    n: int
    nbits: int
    chain: int  # number of successive snapshots
    base_std: float
    seed: int


CONFIGS = {
    "lenet5": Config("lenet5", 61_706, 3, 1, 0.1, SEED0 + 1),
    "resnet18": Config("resnet18", 11_689_512, 4, 10, 0.05, SEED0 + 2),
    "vgg16": Config("vgg16", 138_357_544, 4, 1, 0.02, SEED0 + 3),
    "xfmr1p3b": Config("xfmr1p3b", 1_315_575_808, 5, 4, 0.02, SEED0 + 4),
}


def base_state(cfg: Config, device, n=None):
    return normal(cfg.n if n is None else n, cfg.base_std, device, cfg.seed)


def snapshot_delta(cfg: Config, t: int, device, n=None):
    """The true update u_t - u_{t-1} of snapshot t (1-based) as drawn (before any fp32 re-rounding)."""
    n = cfg.n if n is None else n
    seed = cfg.seed + 1000 * t
    if cfg.name == "lenet5":
        return laplace(n, 1e-3, device, seed)
    if cfg.name == "resnet18":
        # -0.1 * g with g ~ N(0, s_l^2), s_l log-uniform in [1e-4, 1e-2], drawn once per segment.
        gs = _gen("cpu", cfg.seed + 7)
        seg = resnet18_segments()
        s_l = torch.exp(torch.rand(len(seg), generator=gs) * (math.log(1e-2) - math.log(1e-4)) + math.log(1e-4))
        scale = torch.repeat_interleave(s_l, torch.tensor(seg))[:n].to(device)
        return -0.1 * normal(n, 1.0, device, seed) * scale
    if cfg.name == "vgg16":
        d = student_t3(n, 1e-4, device, seed)
        # 20 % of the entries exactly zero, in contiguous blocks (frozen parameters).
        block = 1 << 16
        nblocks = (n + block - 1) // block
        gp = _gen("cpu", cfg.seed + 9)
        frozen = torch.randperm(nblocks, generator=gp)[: nblocks // 5]
        mask = torch.zeros(nblocks, dtype=torch.bool)
        mask[frozen] = True
        mask = torch.repeat_interleave(mask.to(device), block)[:n]
        d[mask] = 0.0
        return d
    if cfg.name == "xfmr1p3b":
        return lognormal_signed(n, 1e-4, 1.5, device, seed)
    raise KeyError(cfg.name)


SWEEP_DISTS = ("gauss", "laplace", "lognormal", "one_exp", "one_exp_2sign", "zero")


def sweep_delta(dist: str, n: int, device, seed):
    if dist == "gauss":
        return normal(n, 1e-3, device, seed)
    if dist == "laplace":
        return laplace(n, 1e-3, device, seed)
    if dist == "lognormal":
        return lognormal_signed(n, 1e-4, 1.5, device, seed)
    if dist == "one_exp":
        return one_exponent(n, -13, device, seed, two_sign=False)
    if dist == "one_exp_2sign":
        return one_exponent(n, -13, device, seed, two_sign=True)
    if dist == "zero":
        return torch.zeros(n, dtype=torch.float32, device=device)
    raise KeyError(dist)
