"""Seeded synthetic inputs shared by the CUDA-path tests, the oracle tests and the benchmark.

This module holds none of the method's arithmetic: it only draws the random tensors the
workloads are defined on.  The paper (arXiv 1801.04928) uses no dataset; the workloads are
fully-connected sigmoid networks of L weight layers, all N wide, on B samples:

    w^l ~ N(0, 1/N)   (std 1/sqrt(N)),   shape [L, N, N], row j = incoming weights of neuron j
    b^l ~ N(0, 1),                        shape [L, N]
    x   ~ U[0, 1),                        shape [B, N]
    y   : one-hot at a seeded index per sample ("onehot") or U[0, 1) ("uniform"), [B, N]

Everything is float32 (the storage type of the library) and comes from one
``torch.Generator`` seeded with ``SEED_BASE + config index`` on the requested device, so the
CUDA path and the oracle (given a host copy) see bit-identical values.
"""
from __future__ import annotations

import torch

SEED_BASE = 18010492800

# The named workloads: index -> sizes, leapfrog worker count and target kind.
CONFIGS = {
    1: dict(L=8, N=64, B=1, k=2, y="onehot"),
    2: dict(L=32, N=1024, B=1, k=4, y="uniform"),
    3: dict(L=64, N=4096, B=1, k=8, y="uniform"),
    4: dict(L=16, N=4096, B=256, k=4, y="onehot"),
}

# The sweep grid (L fixed at 48); B = 1 points use uniform targets, B > 1 one-hot.
SWEEP = dict(L=48, N=(256, 1024, 4096, 8192), B=(1, 16, 128, 1024), k=(1, 2, 4, 8, 16))
SWEEP_CONFIG_INDEX = 5


def make_inputs(L: int, N: int, B: int, y: str = "uniform", seed: int = SEED_BASE,
                device: str | torch.device = "cpu") -> dict[str, torch.Tensor]:
    """Draw w, b, x, y for one workload on ``device`` (float32, contiguous)."""
    if y not in ("onehot", "uniform"):
        raise ValueError("y must be 'onehot' or 'uniform'")
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(int(seed))
    w = torch.empty((L, N, N), dtype=torch.float32, device=dev)
    for l in range(L):  # layer by layer: no temporary larger than one matrix
        w[l].normal_(0.0, 1.0, generator=g).mul_(float(N) ** -0.5)
    b = torch.empty((L, N), dtype=torch.float32, device=dev).normal_(0.0, 1.0, generator=g)
    x = torch.empty((B, N), dtype=torch.float32, device=dev).uniform_(0.0, 1.0, generator=g)
    if y == "uniform":
        yt = torch.empty((B, N), dtype=torch.float32, device=dev).uniform_(0.0, 1.0, generator=g)
    else:
        idx = torch.randint(0, N, (B,), generator=g, device=dev)
        yt = torch.zeros((B, N), dtype=torch.float32, device=dev)
        yt[torch.arange(B, device=dev), idx] = 1.0
    return dict(w=w, b=b, x=x, y=yt)


def make_config(index: int, device: str | torch.device = "cpu", **override):
    """Inputs of a named workload; returns (sizes dict, tensors dict)."""
    cfg = dict(CONFIGS[index])
    cfg.update(override)
    t = make_inputs(cfg["L"], cfg["N"], cfg["B"], cfg["y"], SEED_BASE + index, device)
    return cfg, t


def make_inputs_widths(widths, B: int, y: str = "uniform", seed: int = SEED_BASE,
                       device: str | torch.device = "cpu") -> dict[str, torch.Tensor]:
    """The same distributions for a network whose layers have widths n_0..n_L (w^l is
    n_l x n_{l-1} with std 1/sqrt(n_{l-1})).  Every tensor is flat: the per-layer blocks one after
    the other, in layer order (w: [n_l][n_{l-1}] row-major; b: [n_l]; x: [B][n_0]; y: [B][n_L])."""
    if y not in ("onehot", "uniform"):
        raise ValueError("y must be 'onehot' or 'uniform'")
    n = [int(v) for v in widths]
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(int(seed))
    w = torch.cat([torch.empty(n[l] * n[l - 1], dtype=torch.float32, device=dev)
                   .normal_(0.0, 1.0, generator=g).mul_(float(n[l - 1]) ** -0.5) for l in range(1, len(n))])
    b = torch.empty(sum(n[1:]), dtype=torch.float32, device=dev).normal_(0.0, 1.0, generator=g)
    x = torch.empty(B * n[0], dtype=torch.float32, device=dev).uniform_(0.0, 1.0, generator=g)
    if y == "uniform":
        yt = torch.empty(B * n[-1], dtype=torch.float32, device=dev).uniform_(0.0, 1.0, generator=g)
    else:
        idx = torch.randint(0, n[-1], (B,), generator=g, device=dev)
        yt = torch.zeros((B, n[-1]), dtype=torch.float32, device=dev)
        yt[torch.arange(B, device=dev), idx] = 1.0
        yt = yt.reshape(-1)
    return dict(w=w, b=b, x=x, y=yt)
