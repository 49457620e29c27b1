"""Seeded synthetic inputs shaped like the paper's workloads.

The paper's datasets (its dataset table: Synthetic 10/100/1000, YearPrediction, cadata, cpusmall,
cod-rna, gisette, a 128-projection tomography volume) are not available here; the five workloads
below stand in for their shapes.  This module holds no arithmetic of the method itself: it only
draws A, x*, b = A x* + noise.  The same arrays feed the CUDA path and whatever checks it.

Every generator takes (m, n) overrides so that tests can run reduced sizes with the same
distributions, and a torch device so that full sizes can be drawn directly in device memory.
"""
from dataclasses import dataclass, field
import math

import torch


@dataclass
class Workload:
    name: str
    m: int
    n: int
    bits: int
    batch: int
    lr: float
    epochs: int
    levels: str = "uniform"        # "uniform" | "optimal"
    model_bits: int = 0
    grad_bits: int = 0
    hist_bins: int = 1024
    seed: int = 0
    extra: dict = field(default_factory=dict)


WORKLOADS = {
    "c1": Workload("c1: 4096x64 U[-1,1], 4-bit uniform, B=16", 4096, 64, 4, 16, 0.01, 10),
    "c2": Workload("c2: 100000x1000 clipped N(0,1), 8-bit uniform, B=256", 100_000, 1000, 8, 256, 1e-3, 5),
    "c3": Workload("c3: 1000000x2048 U[-1,1], 2-bit data, 8-bit model and gradient, B=1024",
                   1_000_000, 2048, 2, 1024, 5e-4, 3, model_bits=8, grad_bits=8),
    "c4": Workload("c4: 500000x512 signed lognormal, 3-bit optimal levels, B=512", 500_000, 512, 3, 512, 1e-3, 5,
                   levels="optimal"),
    "c4u": Workload("c4u: 500000x512 signed lognormal, 3-bit uniform levels, B=512", 500_000, 512, 3, 512, 1e-3, 5),
    "c5": Workload("c5: 65536x32768 5% dense tomography rows, 4-bit uniform, B=2048", 65_536, 32_768, 4, 2048,
                   1e-4, 2),
}


def _gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _labels(A, xstar, noise, g, chunk=1 << 16):
    m = A.shape[0]
    b = torch.empty(m, dtype=torch.float32, device=A.device)
    for r0 in range(0, m, chunk):
        r1 = min(m, r0 + chunk)
        clean = (A[r0:r1].double() @ xstar.double())
        b[r0:r1] = (clean + noise * torch.randn(r1 - r0, generator=g, device=A.device, dtype=torch.float64)).float()
    return b


def _fill_rows(m, n, device, fn, chunk_elems=1 << 26):
    A = torch.empty((m, n), dtype=torch.float32, device=device)
    rows = max(1, chunk_elems // n)
    for r0 in range(0, m, rows):
        r1 = min(m, r0 + rows)
        A[r0:r1] = fn(r1 - r0)
    return A


def make(key, m=None, n=None, device="cpu", seed=None):
    """Returns (workload, A (m, n) fp32, b (m,) fp32, xstar (n,) fp32) on `device`."""
    base = WORKLOADS[key]
    w = Workload(**{**base.__dict__})
    if m is not None:
        w.m = int(m)
    if n is not None:
        w.n = int(n)
    if seed is not None:
        w.seed = int(seed)
    m, n = w.m, w.n
    g = _gen(1000 + w.seed, device)
    kind = key[:2]
    if kind == "c1":
        A = _fill_rows(m, n, device, lambda r: torch.rand((r, n), generator=g, device=device) * 2 - 1)
        xstar = torch.randn(n, generator=g, device=device)
        noise = 0.01
    elif kind == "c2":
        A = _fill_rows(m, n, device, lambda r: torch.randn((r, n), generator=g, device=device).clamp_(-3, 3))
        xstar = torch.randn(n, generator=g, device=device) / math.sqrt(n)
        noise = 0.1
    elif kind == "c3":
        A = _fill_rows(m, n, device, lambda r: torch.rand((r, n), generator=g, device=device) * 2 - 1)
        xstar = torch.randn(n, generator=g, device=device) / math.sqrt(n)
        noise = 0.05
    elif kind == "c4":
        def rows(r):
            mag = torch.exp(1.5 * torch.randn((r, n), generator=g, device=device))
            sign = (torch.rand((r, n), generator=g, device=device) < 0.5).float() * 2 - 1
            return mag * sign
        A = _fill_rows(m, n, device, rows)
        A /= A.abs().amax(dim=0, keepdim=True).clamp_min(1e-30)
        xstar = torch.randn(n, generator=g, device=device) / math.sqrt(n)
        noise = 0.05
    elif kind == "c5":
        def rows(r):
            keep = torch.rand((r, n), generator=g, device=device) < 0.05
            return torch.rand((r, n), generator=g, device=device) * keep
        A = _fill_rows(m, n, device, rows, chunk_elems=1 << 25)
        side = int(math.isqrt(n))
        img = torch.rand((side, side), generator=g, device=device)
        sigma, rad = 3.0, 9
        t = torch.arange(-rad, rad + 1, device=device, dtype=torch.float32)
        k1 = torch.exp(-0.5 * (t / sigma) ** 2)
        k1 /= k1.sum()
        img = torch.nn.functional.conv2d(img[None, None], k1.view(1, 1, 1, -1), padding=(0, rad))
        img = torch.nn.functional.conv2d(img, k1.view(1, 1, -1, 1), padding=(rad, 0))[0, 0]
        xstar = torch.zeros(n, device=device)
        xstar[: side * side] = img.flatten()
        noise = 0.01
    else:
        raise KeyError(key)
    b = _labels(A, xstar.float(), noise, g)
    return w, A, b, xstar.float()
