"""Seeded synthetic inputs for the blocked adaptive randomized range finder.

This module only *generates inputs* (test matrices A with a prescribed
spectrum and Gaussian sampling matrices Omega).  It contains none of the
method's arithmetic and is imported by the tests, by the smoke check and by the
benchmark.  The CPU oracle and the CUDA library never import it:
they receive its arrays as arguments, so both sides see the same bytes.

Workloads mirror the paper's experiments: matrices with prescribed singular
values and random orthogonal singular vectors (stability experiment in the
section "Numerical Stability and Performance"), and a GaLore-shaped low-rank
gradient plus noise (section "Towards Efficient Low-Rank Deep Learning").
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Workload:
    """One range-finder problem: shape, spectrum recipe, and stop parameters."""

    name: str
    dtype: str          # "f64" or "f32": arithmetic type of the GPU path
    m: int
    n: int
    b: int              # block size
    tol: float          # relative Frobenius tolerance
    max_rank: int
    kind: str           # spectrum recipe, see sigma()
    seed: int
    rank: int = 0       # number of non-trivial singular triplets built (0: min(m, n))
    noise_std: float = 0.0

    def scaled(self, m: int, n: int, max_rank: int | None = None, b: int | None = None,
               rank: int | None = None, name: str | None = None) -> "Workload":
        """Same recipe at another size (parity-test cases)."""
        return dataclasses.replace(
            self, m=m, n=n,
            max_rank=self.max_rank if max_rank is None else max_rank,
            b=self.b if b is None else b,
            rank=self.rank if rank is None else rank,
            name=name or f"{self.name}_{m}x{n}")

    @property
    def np_dtype(self):
        return np.float64 if self.dtype == "f64" else np.float32


# The five benchmark configurations (index 0..4) and the second reading of the
# fourth one's noise level ("cfg4b": 1e-6 taken as a standard deviation).
CONFIGS = {
    "cfg1": Workload("cfg1", "f64", 1024, 768, 16, 1e-8, 256, "exp20", 1001),
    "cfg2": Workload("cfg2", "f64", 8192, 8192, 64, 1e-4, 1024, "poly2", 1002),
    "cfg3": Workload("cfg3", "f64", 4096, 4096, 32, 1e-13, 768, "stress", 1003),
    "cfg4": Workload("cfg4", "f32", 4096, 11008, 64, 1e-2, 512, "galore", 1004,
                     rank=128, noise_std=1e-3),
    "cfg4b": Workload("cfg4b", "f32", 4096, 11008, 64, 1e-2, 512, "galore", 1004,
                      rank=128, noise_std=1e-6),
    "cfg5": Workload("cfg5", "f64", 32768, 16384, 128, 1e-6, 2048, "exp150", 1005, rank=2048),
}


def sigma(w: Workload) -> np.ndarray | None:
    """Prescribed singular values (descending), or None when the recipe has none."""
    p = min(w.m, w.n)
    r = p if w.rank == 0 else min(w.rank, p)
    j = np.arange(1, r + 1, dtype=np.float64)
    if w.kind == "exp20":
        s = np.exp(-(j - 1.0) / 20.0)
    elif w.kind == "poly2":
        s = j ** -2.0
    elif w.kind == "stress":
        # log-uniform decay over 15 decades across the first 512 values, then a 1e-16 floor;
        # at reduced sizes the 15 decades are compressed onto the first p/8 values.
        knee = 512 if p >= 4096 else max(2, p // 8)
        s = np.where(j <= knee, 10.0 ** (-15.0 * (j - 1.0) / (knee - 1.0)), 1e-16)
    elif w.kind == "exp150":
        s = np.exp(-j / 150.0)
    elif w.kind == "galore":
        return None
    else:
        raise ValueError(f"unknown spectrum recipe {w.kind!r}")
    return s


def _haar(rng: np.random.Generator, rows: int, cols: int) -> np.ndarray:
    """Orthonormal columns: thin Q factor of a Householder QR of a Gaussian matrix."""
    q, _ = np.linalg.qr(rng.standard_normal((rows, cols)))
    return q


def make_matrix(w: Workload, device: str | None = None):
    """Build A for workload `w`.

    Returns (A, sigma) with A a numpy array of w.np_dtype, or, if `device` is a
    torch device string, a torch tensor on that device (the large product
    U diag(sigma) V^T is then formed there; this is input generation only).
    """
    rng = np.random.default_rng(w.seed)
    if w.kind == "galore":
        r = w.rank
        g1 = rng.standard_normal((w.m, r)) / np.sqrt(128.0)
        g2 = rng.standard_normal((w.n, r)) / np.sqrt(128.0)
        if device is None:
            a = g1 @ g2.T
            a += w.noise_std * rng.standard_normal((w.m, w.n))
            return a.astype(w.np_dtype), None
        import torch
        a = torch.from_numpy(g1).to(device) @ torch.from_numpy(g2).to(device).T
        noise = rng.standard_normal((w.m, w.n), dtype=np.float32)
        a += w.noise_std * torch.from_numpy(noise).to(device).to(torch.float64)
        return a.to(torch.float64 if w.dtype == "f64" else torch.float32).contiguous(), None

    s = sigma(w)
    r = s.shape[0]
    u = _haar(rng, w.m, r)
    v = _haar(rng, w.n, r)
    if device is None:
        a = (u * s) @ v.T
        return a.astype(w.np_dtype), s
    import torch
    ut = torch.from_numpy(u).to(device)
    vt = torch.from_numpy(v).to(device)
    a = (ut * torch.from_numpy(s).to(device)) @ vt.T
    return a.to(torch.float64 if w.dtype == "f64" else torch.float32).contiguous(), s


def make_omega(w: Workload) -> np.ndarray:
    """Gaussian sampling matrix Omega (n x max_rank), column block i = Omega_i.

    Drawn from the workload's seed on a stream separate from A's, as float64;
    callers round to the path's dtype.
    """
    rng = np.random.default_rng([w.seed, 7])
    return rng.standard_normal((w.n, w.max_rank))


def diag_matrix(s: np.ndarray, m: int, n: int) -> np.ndarray:
    """A = diag(s) padded to m x n (cheap stand-in with the same spectrum)."""
    a = np.zeros((m, n))
    k = min(len(s), m, n)
    a[np.arange(k), np.arange(k)] = s[:k]
    return a
