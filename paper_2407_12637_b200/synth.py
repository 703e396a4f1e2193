"""Seeded synthetic inputs (no arithmetic of the method lives here).

Gradients follow what arXiv 2407.12637 says about them (Sec. 3.3: zero-centred,
a very long tail, sparse around the tail): a Laplace or Student-t body with a
small fraction of entries multiplied by a large factor.  Weights / activations
are raw code bytes, uniformly random, which each consumer decodes itself.

Host flavour: numpy (`np.random.Philox` bit generator).  Device flavour: torch
ops under a seeded `torch.Generator`; a tensor generated on the device is
copied to the host when a CPU check needs the same bytes.
"""
from __future__ import annotations

import numpy as np

OUTLIER_FRACTION = 1e-3
OUTLIER_FACTOR = 50.0


def _rng(seed: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed & (2**64 - 1), stream]))


def laplace_outliers(n: int, scale: float, seed: int, stream: int = 0) -> np.ndarray:
    """fp32 Laplace(0, scale) by inverse CDF; OUTLIER_FRACTION of entries times OUTLIER_FACTOR."""
    r = _rng(seed, stream)
    u = r.random(n) - 0.5
    g = -scale * np.sign(u) * np.log1p(-2.0 * np.abs(u))
    mask = r.random(n) < OUTLIER_FRACTION
    g[mask] *= OUTLIER_FACTOR
    return g.astype(np.float32)


def student_t3(n: int, std: float, seed: int, stream: int = 0) -> np.ndarray:
    """fp32 Student-t with 3 degrees of freedom scaled to standard deviation `std`
    (the variance of t_3 is 3)."""
    r = _rng(seed, stream)
    z = r.standard_normal(n)
    chi = (r.standard_normal((3, n)) ** 2).sum(axis=0) / 3.0
    return (z / np.sqrt(chi) * (std / np.sqrt(3.0))).astype(np.float32)


def code_bytes(nbytes: int, seed: int, stream: int = 0) -> np.ndarray:
    """Uniformly random bytes: two uniform 4-bit codes per byte (signed [-8,7] or unsigned
    [0,15] according to how the consumer reads them)."""
    return _rng(seed, stream).integers(0, 256, size=nbytes, dtype=np.uint8)


def lognormal_walk(steps: int, sigma: float, seed: int, stream: int = 0) -> np.ndarray:
    """Multiplicative random walk of a layer's gradient scale: m_0 = 1,
    m_{t+1} = m_t exp(sigma xi_t), xi ~ N(0, 1)."""
    xi = _rng(seed, stream).standard_normal(max(steps - 1, 0))
    return np.concatenate([[1.0], np.exp(sigma * np.cumsum(xi))])


# ----------------------------------------------------------------------------- device flavour
def _torch_gen(device, seed: int, stream: int):
    import torch
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + stream) & (2**63 - 1))
    return g


def laplace_outliers_torch(n: int, scale: float, seed: int, stream: int = 0, device="cuda"):
    """Device flavour of `laplace_outliers` (same recipe, torch's generator)."""
    import torch
    gen = _torch_gen(device, seed, stream)
    u = torch.rand(n, generator=gen, device=device, dtype=torch.float32) - 0.5
    g = -scale * torch.sign(u) * torch.log1p(-2.0 * u.abs())
    u.uniform_(0.0, 1.0, generator=gen)
    g = torch.where(u < OUTLIER_FRACTION, g * OUTLIER_FACTOR, g)
    return torch.nan_to_num_(g, nan=0.0, posinf=scale * 20.0, neginf=-scale * 20.0)


def student_t3_torch(n: int, std: float, seed: int, stream: int = 0, device="cuda"):
    """Device flavour of `student_t3`."""
    import torch
    gen = _torch_gen(device, seed, stream)
    z = torch.randn(n, generator=gen, device=device, dtype=torch.float32)
    chi = torch.zeros(n, device=device, dtype=torch.float32)
    for _ in range(3):
        chi += torch.randn(n, generator=gen, device=device, dtype=torch.float32) ** 2
    chi.div_(3.0).clamp_(min=1e-12)
    return z / chi.sqrt() * (std / 3.0 ** 0.5)


def code_bytes_torch(nbytes: int, seed: int, stream: int = 0, device="cuda"):
    """Device flavour of `code_bytes`."""
    import torch
    gen = _torch_gen(device, seed, stream)
    return torch.randint(0, 256, (nbytes,), generator=gen, device=device, dtype=torch.uint8)
