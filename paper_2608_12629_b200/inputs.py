"""Seeded synthetic K-means inputs shared by the tests, the oracle harness and the benchmark.

This module holds NO K-means arithmetic (no distances, no means): it only draws Gaussian-mixture
points, rounds them once to bf16 and samples initial centroids, so that the CUDA path and the CPU
oracle can be fed the very same bits.  The mixtures stand in for the paper's Sparse-VideoGen2 token
features (Section 5, "Flash-KMeans clean-start workload"), which are not available; the shapes
follow the paper's B=32 / N=65,536 / K=1,024 / D=128 family.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int            # independent problems
    N: int            # points per problem
    D: int            # features
    K: int            # clusters
    components: int   # mixture components
    mean_std: float   # component means ~ N(0, mean_std^2 I)
    sigma: float      # per-coordinate std of each component
    weights: str      # "uniform" | "dirichlet"
    iters: int
    seed: int


WORKLOADS = {
    # small case the oracle finishes in seconds
    "c1": Workload("c1", 1, 32768, 64, 128, 128, 2.0, 1.0, "uniform", 10, 1001),
    # the configuration the headline metric is quoted on
    "c2": Workload("c2", 1, 1048576, 128, 1024, 1024, 1.0, 0.5, "uniform", 20, 1002),
    # batched independent problems, unequal component weights
    "c3": Workload("c3", 32, 65536, 128, 256, 256, 1.0, 0.5, "dirichlet", 10, 1003),
    # large K: many sparse or empty clusters
    "c4": Workload("c4", 1, 2097152, 256, 65536, 16384, 1.0, 0.3, "uniform", 5, 1004),
    # few clusters, one problem: the shape class of the single-pass (fused) iteration, X larger than L2
    "f1": Workload("f1", 1, 2097152, 64, 64, 64, 1.0, 0.5, "uniform", 10, 1006),
    # rows of 1,024 features: no X tile stays resident, the contraction is streamed over D
    "w1": Workload("w1", 1, 262144, 1024, 1024, 1024, 1.0, 0.5, "uniform", 5, 1007),
    # the paper's own clean-start shape (assign only in the paper)
    "paper": Workload("paper", 32, 65536, 128, 1024, 1024, 1.0, 0.5, "uniform", 3, 1005),
}


def sweep_workload(N: int, D: int, K: int, iters: int = 3) -> Workload:
    """One shape of the shape sweep: min(K, 16384) components, means ~ N(0,I), sigma 0.5."""
    seed = 2000 + (N * 1315423911 + D * 2654435761 + K * 97) % 100000
    return Workload(f"sweep_n{N}_d{D}_k{K}", 1, N, D, K, min(K, 16384), 1.0, 0.5, "uniform", iters, seed)


def gaussian_mixture(N: int, D: int, components: int, mean_std: float, sigma: float, seed: int,
                     weights: str = "uniform", device: str | torch.device = "cpu",
                     chunk: int = 1 << 18):
    """Draw N points of a `components`-component isotropic Gaussian mixture, rounded once to bf16.

    Returns (X bf16 [N,D], labels int64 [N]) on `device`.  fp32 math, one RNE cast.  The stream of
    random numbers depends on the device type, so a test must generate on one device and copy.
    """
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(int(seed))
    means = torch.randn(components, D, generator=g, device=dev, dtype=torch.float32) * mean_std
    if weights == "uniform":
        labels = torch.randint(0, components, (N,), generator=g, device=dev)
    elif weights == "dirichlet":
        # Dirichlet(1) = normalised Exp(1) draws
        u = torch.rand(components, generator=g, device=dev, dtype=torch.float32).clamp_min(1e-12)
        w = -torch.log(u)
        w = w / w.sum()
        labels = torch.multinomial(w, N, replacement=True, generator=g)
    else:
        raise ValueError(weights)
    X = torch.empty(N, D, device=dev, dtype=torch.bfloat16)
    for s in range(0, N, chunk):
        e = min(N, s + chunk)
        noise = torch.randn(e - s, D, generator=g, device=dev, dtype=torch.float32)
        X[s:e] = (means[labels[s:e]] + sigma * noise).to(torch.bfloat16)
    return X, labels


def sample_init(X: torch.Tensor, K: int, seed: int) -> torch.Tensor:
    """C0 = K distinct rows of X (random sample without replacement), bf16 [K,D]."""
    g = torch.Generator(device=X.device)
    g.manual_seed(int(seed) + 7919)
    N = X.shape[0]
    if K <= N:
        rows = torch.randperm(N, generator=g, device=X.device)[:K]
    else:  # more clusters than points: rows repeat
        rows = torch.randint(0, N, (K,), generator=g, device=X.device)
    return X[rows].contiguous()


def make_problem(w: Workload, device: str | torch.device = "cpu", b: int = 0):
    """Problem `b` of workload `w`: (X bf16 [N,D], C0 bf16 [K,D])."""
    X, _ = gaussian_mixture(w.N, w.D, w.components, w.mean_std, w.sigma, w.seed + b, w.weights, device)
    return X, sample_init(X, w.K, w.seed + b)


def make_batch(w: Workload, device: str | torch.device = "cpu"):
    """All problems of `w`: (X bf16 [B,N,D], C0 bf16 [B,K,D])."""
    Xs, Cs = zip(*(make_problem(w, device, b) for b in range(w.B)))
    return torch.stack(Xs).contiguous(), torch.stack(Cs).contiguous()


def to_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 array of its raw bits (host copy)."""
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def from_bits(a: np.ndarray, device: str | torch.device = "cpu") -> torch.Tensor:
    """numpy uint16 bf16 bits -> bf16 tensor."""
    a = np.ascontiguousarray(a, dtype=np.uint16)
    return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).to(device)


def checksum(t: torch.Tensor) -> int:
    """64-bit checksum of a bf16 tensor's raw bits (logged beside every measured number)."""
    v = t.detach().contiguous().view(torch.int16).to(torch.int64) & 0xFFFF
    idx = torch.arange(v.numel(), device=v.device, dtype=torch.int64).view(v.shape)
    return int(((v * 2654435761 + idx * 40503) & 0x7FFFFFFF).sum().item()) & 0xFFFFFFFFFFFFFFFF
