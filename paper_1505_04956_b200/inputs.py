"""Seeded synthetic inputs: Gaussian-mixture sample matrices and initial centres.

This module only draws random inputs.  It contains none of the method's arithmetic (no distances,
no assignment, no gradient), so the same buffers can be handed to the CUDA library and to any
independent check of it.

The recipe follows the paper's description of its synthetic data (Section 5.3, "Synthetic Data
Sets"): pick k cluster centres at random, then draw every sample from the distribution that belongs
to one of the centres.  Here that is: component means from a box or a Gaussian, mixture weights
equal or Dirichlet(1), each row = mean[component] + sigma * N(0, I), fp32, row-major.
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    """One K-Means ASGD workload: data shape, mixture recipe and the optimiser's parameters."""
    name: str
    N: int
    d: int
    k: int
    W: int
    b: int
    eps: float
    steps: int                 # steps per worker (0 = `passes` full passes over the shard)
    passes: int
    comm_interval: int
    fanout: int
    seed: int
    means: str                 # "box:<half-width>" or "normal:<std>"
    sigma: float
    weights: str               # "equal" or "dirichlet"
    components: Optional[int] = None   # mixture components (default k)

    @property
    def H(self) -> int:
        return self.N // self.W

    @property
    def B(self) -> int:
        return self.H // self.b

    def steps_per_worker(self) -> int:
        return self.steps if self.steps > 0 else self.passes * self.B

    def scaled(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The workloads the library is measured and tested on: five base shapes and the large-codebook shape
# (k = 1000 prototypes of d = 128, the top of the codebook range of Section 5.2).
WORKLOADS = {
    "tiny": Workload("tiny", 100_000, 10, 10, 4, 100, 0.05, 1000, 0, 10, 1, 0, "box:10", 1.0, "equal"),
    "stream": Workload("stream", 268_435_456, 10, 10, 592, 500, 0.01, 0, 1, 20, 1, 1, "box:10", 1.0, "equal"),
    "mid": Workload("mid", 16_777_216, 128, 100, 296, 1000, 0.01, 0, 2, 10, 2, 2, "normal:5", 1.0, "dirichlet"),
    "sweep": Workload("sweep", 67_108_864, 32, 64, 592, 256, 0.02, 0, 1, 10, 1, 3, "box:5", 0.5, "equal"),
    "dense": Workload("dense", 8_388_608, 256, 1024, 148, 4096, 0.005, 0, 1, 5, 1, 4, "normal:2", 1.0, "equal"),
    "codebook": Workload("codebook", 8_388_608, 128, 1000, 148, 2048, 0.005, 0, 1, 5, 1, 5, "normal:3", 1.0, "equal"),
}


def mixture_parameters(wl: Workload, device="cpu"):
    """Component means [C, d] and mixture weights [C], drawn on the CPU generator from wl.seed."""
    g = torch.Generator(device="cpu")
    g.manual_seed(1_000_003 * wl.seed + 17)
    C = wl.components or wl.k
    kind, val = wl.means.split(":")
    if kind == "box":
        mu = (torch.rand(C, wl.d, generator=g, dtype=torch.float64) * 2 - 1) * float(val)
    elif kind == "normal":
        mu = torch.randn(C, wl.d, generator=g, dtype=torch.float64) * float(val)
    else:
        raise ValueError(wl.means)
    if wl.weights == "equal":
        p = torch.full((C,), 1.0 / C, dtype=torch.float64)
    elif wl.weights == "dirichlet":
        e = -torch.log(torch.rand(C, generator=g, dtype=torch.float64).clamp_min(1e-300))
        p = e / e.sum()
    else:
        raise ValueError(wl.weights)
    return mu.to(torch.float32).to(device), p.to(device)


def make_samples(wl: Workload, device="cpu", rows: Optional[int] = None, chunk: int = 1 << 22):
    """X [rows or wl.N, d] fp32 on `device`, generated chunk by chunk with that device's generator.

    Returns (X, component_means).  The values depend on the device kind and the torch version, so a
    check that needs the same numbers on the host copies this very buffer.
    """
    n = int(rows if rows is not None else wl.N)
    dev = torch.device(device)
    mu, p = mixture_parameters(wl, dev)
    g = torch.Generator(device=dev)
    g.manual_seed(wl.seed)
    X = torch.empty((n, wl.d), dtype=torch.float32, device=dev)
    cdf = torch.cumsum(p, 0)
    cdf[-1] = 1.0
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        u = torch.rand(hi - lo, generator=g, device=dev, dtype=torch.float64)
        comp = torch.searchsorted(cdf, u).clamp_max(mu.shape[0] - 1)
        del u
        out = X[lo:hi]
        out.normal_(0.0, wl.sigma, generator=g)
        out += mu[comp]
        del comp
    return X, mu


def initial_centres(wl: Workload, X: torch.Tensor):
    """w0 [k, d]: k distinct seeded-random rows of X (the control thread's problem-dependent w0)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(7_919 * wl.seed + 3)
    n = X.shape[0]
    chosen = []
    seen = set()
    while len(chosen) < wl.k:
        r = int(torch.randint(0, n, (1,), generator=g))
        if r not in seen:
            seen.add(r)
            chosen.append(r)
    idx = torch.tensor(chosen, dtype=torch.long, device=X.device)
    return X.index_select(0, idx).contiguous()
