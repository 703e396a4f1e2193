"""Pins for the oracle's clipping-factor update (Eq. 14-16, Algorithm 1) -- CPU only."""
import os

import numpy as np
import pytest

from oracle import analysis, ref
from paper_2407_12637_b200 import synth
from test_oracle_quantizer import CF


def _iterate(g, bits, alpha, beta, steps, gamma0=1.0, gamma_min=None):
    gm, _ = ref.grad_stats(g)
    gamma = np.float32(gamma0)
    traj = [gamma]
    for _ in range(steps):
        n_out = ref.clip_count(g, gamma * gm)
        gamma = ref.update_interval(gamma, alpha, beta, beta if gamma_min is None else gamma_min,
                                    1.0, bits, g.size, n_out)
        traj.append(gamma)
    return np.array(traj, np.float32), gm


def test_sign_cases():
    # R_out - alpha/(2^b-1): n_out*(2^b-1) versus alpha*N; alpha = 2^-10 is exact in binary32
    alpha, n = 2.0 ** -10, 15 * 1024
    assert ref.update_sign(4, alpha, n, 1) == 0          # 1*15 == 15
    assert ref.update_sign(4, alpha, n, 2) == 1
    assert ref.update_sign(4, alpha, n, 0) == -1
    assert ref.update_sign(8, alpha, 255 * 1024, 1) == 0
    assert ref.update_sign(8, alpha, 255 * 1024 + 1, 1) == -1


def test_one_step_follows_eq15():
    beta = np.float32(1e-3)
    g0 = np.float32(0.5)
    assert ref.update_interval(g0, 1e-3, beta, beta, 1.0, 4, 10**6, 10**5) == np.float32(g0 + beta)
    assert ref.update_interval(g0, 1e-3, beta, beta, 1.0, 4, 10**6, 0) == np.float32(g0 - beta)
    assert ref.update_interval(g0, 2.0 ** -10, beta, beta, 1.0, 4, 15 * 1024, 1) == g0   # sign(0) = 0
    assert ref.update_interval(1.0, 1e-3, beta, beta, 1.0, 4, 10**6, 10**5) == np.float32(1.0)  # clamp
    assert ref.update_interval(beta, 1e-3, beta, beta, 1.0, 4, 10**6, 0) == beta                # clamp
    assert ref.update_interval(g0, 1e-3, beta, beta, 1.0, 4, 10**6, 10**5, n_nonfinite=1) == g0
    assert ref.update_interval(g0, 1e-3, 0.0, 0.0, 1.0, 4, 10**6, 10**5) == g0   # beta = 0: fixed gamma


@pytest.mark.parametrize("bits", [4, 6, 8])
def test_fixed_point_brackets_eq14(bits):
    """On a frozen gradient the iteration settles where R_out brackets alpha/(2^b-1), Eq. (14)."""
    g = synth.laplace_outliers(1 << 17, 1e-3, seed=2)
    alpha, beta = 1e-2, np.float32(1.0 / 64)
    traj, gm = _iterate(g, bits, alpha, beta, 200)
    tail = traj[-8:]
    assert tail.max() - tail.min() <= 2 * beta * (1 + 1e-6)        # a fixed point or a 2-cycle
    lo, hi = np.float32(tail.min()), np.float32(tail.max())
    target = CF[bits]["r_out"] * alpha                              # Eq. (14)
    r_hi = ref.clip_count(g, np.float32(hi + beta) * gm) / g.size
    r_lo = ref.clip_count(g, np.float32(max(lo - beta, 0)) * gm) / g.size
    assert r_hi <= target <= r_lo
    # and R_in = alpha - R_out approaches (2^b-2)/(2^b-1) alpha from the matching side
    assert alpha - r_lo <= CF[bits]["r_in"] * alpha <= alpha - r_hi


def test_lower_bit_width_gives_lower_gamma():
    """Supplement S3: the clipping factor settles lower for fewer bits."""
    g = synth.laplace_outliers(1 << 17, 1e-3, seed=4)
    t4, _ = _iterate(g, 4, 1e-2, 1.0 / 128, 300)
    t8, _ = _iterate(g, 8, 1e-2, 1.0 / 128, 300)
    assert t4[-4:].mean() < t8[-4:].mean()


def test_sparser_tail_gives_smaller_gamma():
    """Sec. 4.3: gradients concentrated near zero with a broad sparse tail prefer a small factor."""
    dense = np.random.default_rng(0).uniform(-1, 1, 1 << 16).astype(np.float32)
    sparse = synth.laplace_outliers(1 << 16, 1e-3, seed=6)
    td, _ = _iterate(dense, 4, 1e-2, 1.0 / 128, 300)
    ts, _ = _iterate(sparse, 4, 1e-2, 1.0 / 128, 300)
    assert ts[-4:].mean() < td[-4:].mean()


def test_count_shortcut_has_the_sign_of_the_literal_rule():
    """sign(T) from the plain count #{|g| > c} equals the one from N(G_out) = |G_L beyond c|."""
    rng = np.random.default_rng(3)
    for trial in range(40):
        n = int(rng.integers(20000, 60000))
        g = synth.laplace_outliers(n, 1e-3, seed=100 + trial)
        gm, _ = ref.grad_stats(g)
        alpha = float(rng.choice([1e-3, 5e-3, 2e-2]))
        gamma = np.float32(rng.uniform(0.02, 1.0))
        bits = int(rng.choice([2, 4, 6, 8]))
        n_out = ref.clip_count(g, gamma * gm)
        assert ref.update_sign(bits, alpha, n, n_out) == \
            analysis.literal_update_sign(g, alpha, float(gamma), bits)


def test_unclamped_rule_self_corrects_above_one():
    g = synth.laplace_outliers(1 << 12, 1e-3, seed=8)
    gm, _ = ref.grad_stats(g)
    gamma = np.float32(1.0)
    n_out = ref.clip_count(g, gamma * gm)
    assert n_out == 0
    nxt = ref.update_interval(gamma, 1e-3, 1e-3, 1e-3, np.inf, 4, g.size, n_out)
    assert nxt == np.float32(np.float32(1.0) - np.float32(1e-3))
