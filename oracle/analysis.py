"""Sort-based error metrics of arXiv 2407.12637, Sec. 3.2-3.3 (TEST INFRASTRUCTURE).

Binary64 numpy, written from the definitions: the large-gradient set G_L
(top alpha fraction by magnitude), its clip-in / clip-out split, the
quantization errors E(G), E(G_L) (Eq. 5-7), the upper bound U(G_L) (Eq. 8)
and the ratios R_in, R_out (Eq. 9, 10).  Used only to check the oracle's
quantizer and update rule against what the paper states about them.
"""
from __future__ import annotations

import dataclasses

import numpy as np


@dataclasses.dataclass
class LargeGradientReport:
    n: int                # N(G)
    n_large: int          # N(G_L) = round(alpha N)
    n_in: int             # N(G_in, gamma)
    n_out: int            # N(G_out, gamma)
    r_in: float           # Eq. (9)
    r_out: float          # Eq. (9)
    e_all: float          # E(G),   Eq. (5)
    e_large: float        # E(G_L), Eq. (6) = Eq. (7)
    e_large_in: float     # clip-in part of the numerator of Eq. (7), / (N(G_L) g_max)
    e_large_out: float    # clip-out part
    u_large: float        # U(G_L), Eq. (8)


def large_gradient_report(g, q_g, alpha: float, gamma: float, bits: int, c=None) -> LargeGradientReport:
    """g: full-precision gradients; q_g: their dequantised values Q(g); both any shape.
    N(G_L) = alpha N rounded to the nearest integer (halves to even); among gradients of equal
    magnitude the earlier ones (memory order) enter G_L first.  `c`: the clipping value the quantizer
    used (its binary32 gamma * g_max); by default gamma * g_max in binary64."""
    g = np.asarray(g, np.float64).ravel()
    qg = np.asarray(q_g, np.float64).ravel()
    n = g.size
    mag = np.abs(g)
    g_max = mag.max()
    n_large = int(round(alpha * n))
    order = np.argsort(-mag, kind="stable")          # descending magnitude
    large = order[:n_large]                          # G_L: the top alpha fraction (Sec. 3.2)
    c = gamma * g_max if c is None else float(c)
    out_mask = mag[large] > c                        # G_out (Sec. 3.3)
    n_out = int(out_mask.sum())
    n_in = n_large - n_out
    err = np.abs(g - qg)
    e_all = err.sum() / (n * g_max)                                  # Eq. (5)
    denom = n_large * g_max if n_large else 1.0
    e_in = err[large][~out_mask].sum() / denom                       # Eq. (7), first sum
    e_out = err[large][out_mask].sum() / denom                       # Eq. (7), second sum
    r_in, r_out = n_in / n, n_out / n                                # Eq. (9)
    a = r_in + r_out                                                 # Eq. (10)
    u = ((gamma / (2 ** bits - 2)) * r_in + (1 - gamma) * r_out) / a if a else 0.0   # Eq. (8)
    return LargeGradientReport(n, n_large, n_in, n_out, r_in, r_out, e_all,
                               e_in + e_out, e_in, e_out, u)


def literal_update_sign(g, alpha: float, gamma: float, bits: int) -> int:
    """sign(T) of Eq. (16) with G_out taken literally as the members of G_L beyond the
    clipping value: N(G_out) = min(#{|g| > c}, N(G_L)); compared without division."""
    g32 = np.asarray(g, np.float32).ravel()
    n = g32.size
    mag = np.abs(g32)
    c = np.float32(gamma) * mag.max()                # binary32 product, as the quantizer forms it
    n_clip = int((mag > c).sum())
    n_large = int(round(float(np.float32(alpha)) * n))
    n_gout = min(n_clip, n_large)
    lhs = n_gout * (2 ** bits - 1)
    rhs = float(np.float32(alpha)) * n
    return (lhs > rhs) - (lhs < rhs)
