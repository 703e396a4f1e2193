"""Pins for the oracle's statistics and gradient quantizer (CPU only).

What fixes the expected values: closed forms printed in the paper (Eq. 1-4, the step size and
the two error bounds of Sec. 3.3), invariants (power-of-two scaling, permutation), special
cases, and brute force over exact rationals.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import analysis, ref
from paper_2407_12637_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_closed_forms.txt")


def _closed_forms():
    rows = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        rows[int(f[0])] = dict(levels=int(f[1]), qmax=int(f[2]), step=float(f[3]),
                               u_in=float(f[4]), r_out=float(f[5]), r_in=float(f[6]))
    return rows


CF = _closed_forms()


def _grad(n=1 << 16, seed=3, scale=1e-3):
    return synth.laplace_outliers(n, scale, seed)


# ------------------------------------------------------------------ statistics
def test_absmax_matches_library_and_is_order_free():
    g = _grad()
    gm, bad = ref.grad_stats(g)
    assert bad == 0 and gm == np.abs(g).max()
    p = np.random.default_rng(0).permutation(g.size)
    assert ref.grad_stats(g[p])[0] == gm


def test_absmax_skips_and_counts_nonfinite():
    g = _grad(1000)
    g[[3, 500]] = [np.nan, -np.inf]
    gm, bad = ref.grad_stats(g)
    assert bad == 2
    assert gm == np.abs(g[np.isfinite(g)]).max()


def test_clip_count_brute_force_and_monotone():
    g = _grad()
    gm, _ = ref.grad_stats(g)
    last = None
    for gamma in np.linspace(0.05, 1.0, 20, dtype=np.float32):
        c = np.float32(gamma) * gm
        cnt = ref.clip_count(g, c)
        assert cnt == sum(1 for v in g if abs(float(v)) > float(c))
        if last is not None:
            assert cnt <= last                      # R_out does not grow with gamma (Sec. 3.3)
        last = cnt
    assert ref.clip_count(g, gm) == 0               # gamma = 1 clips nothing


# ------------------------------------------------------------------ quantizer, nearest rounding
@pytest.mark.parametrize("bits", [2, 4, 5, 6, 8])
def test_grid_points_map_to_their_code(bits):
    """g = k * c / qmax is a grid point of Eq. (4): its code is k whenever the division is exact."""
    qmax = CF[bits]["qmax"]
    c = np.float32(qmax * 2.0 ** -10)               # s = 2^-10 exactly
    ks = np.arange(-qmax, qmax + 1)
    g = (ks * 2.0 ** -10).astype(np.float32)
    q = ref.quantize_grad(g, gamma=1.0, g_max=c, bits=bits)
    assert q.scale == np.float32(2.0 ** -10) and q.c == c
    assert list(q.codes) == list(ks)
    assert q.n_out == 0
    assert np.array_equal(ref.dequantize(q.codes, q.scale), g)


@pytest.mark.parametrize("bits", [2, 4, 6, 8])
@pytest.mark.parametrize("gamma", [1.0, 0.6, 0.25])
def test_code_range_and_error_bounds(bits, gamma):
    """Codes stay in [-qmax, qmax]; clip-in error <= gamma g_max / (2^b - 2), the half step;
    clip-out error = |g| - c <= (1 - gamma) g_max (Sec. 3.3, supplement S1)."""
    g = _grad(1 << 15, seed=bits)
    gm, _ = ref.grad_stats(g)
    q = ref.quantize_grad(g, gamma, gm, bits)
    qmax = CF[bits]["qmax"]
    assert q.codes.min() >= -qmax and q.codes.max() <= qmax
    g64 = g.astype(np.float64)
    c, s = float(q.c), float(q.scale)
    # the step of Eq. (2) equals the paper's 2 gamma g_max / (2^b - 2)
    assert s == pytest.approx(CF[bits]["step"] * gamma * float(gm), rel=1e-6)
    err = np.abs(g64 - s * q.codes.astype(np.float64))
    inside = np.abs(g64) <= c
    u_in = CF[bits]["u_in"] * gamma * float(gm)
    assert err[inside].max() <= u_in * (1 + 1e-5)
    out = ~inside
    assert q.n_out == int(out.sum())
    if out.any():
        assert np.all(np.abs(q.codes[out]) == qmax)
        assert np.allclose(err[out], np.abs(g64[out]) - qmax * s, rtol=0, atol=1e-6 * float(gm))
        assert err[out].max() <= (1 - gamma) * float(gm) * (1 + 1e-5) + 1e-6 * float(gm)


def test_two_bit_quantizer_is_ternary():
    g = _grad(4096)
    gm, _ = ref.grad_stats(g)
    q = ref.quantize_grad(g, 1.0, gm, 2)
    assert set(np.unique(q.codes)) <= {-1, 0, 1}
    assert np.array_equal(q.codes, np.where(np.abs(g) > gm / 2, np.sign(g), 0).astype(np.int8))


def test_nearest_against_exact_rationals():
    """Brute force: the code is the integer nearest to fl32(g / s) (ties to even), evaluated
    over exact rationals of the binary32 operands."""
    rng = np.random.default_rng(7)
    g = (rng.standard_normal(3000) * 1e-3).astype(np.float32)
    g[:16] = np.float32(0.0)
    gm, _ = ref.grad_stats(g)
    for bits, gamma in [(4, 0.7), (6, 1.0), (8, 0.33)]:
        q = ref.quantize_grad(g, gamma, gm, bits)
        qmax = CF[bits]["qmax"]
        s = Fraction(float(q.scale))
        for gi, code in zip(g, q.codes):
            x = np.float32(gi) / q.scale            # one binary32 division, Eq. (1)
            x = Fraction(float(min(max(x, np.float32(-qmax)), np.float32(qmax))))
            fl = x.numerator // x.denominator
            r = x - fl
            want = fl + (1 if r > Fraction(1, 2) or (r == Fraction(1, 2) and fl % 2) else 0)
            assert code == want
            # and that integer really is nearest to the exact quotient, within a binary32 ulp of x
            exact = Fraction(float(gi)) / s
            if abs(exact) <= qmax:
                assert abs(exact - code) <= Fraction(1, 2) + abs(exact) * Fraction(1, 2**23)


def test_power_of_two_scale_invariance():
    """Scaling dY by 2^k scales g_max, c, s by exactly 2^k and leaves codes and n_out alone."""
    g = _grad(1 << 14, seed=11)
    gm, _ = ref.grad_stats(g)
    for rounding in (0, 1):
        base = ref.quantize_grad(g, 0.37, gm, 4, rounding, seed=9, it=2)
        for k in (-7, 5, 20):
            f = np.float32(2.0 ** k)
            gm2, _ = ref.grad_stats(g * f)
            assert gm2 == gm * f
            q2 = ref.quantize_grad(g * f, 0.37, gm2, 4, rounding, seed=9, it=2)
            assert q2.c == base.c * f and q2.scale == base.scale * f
            assert np.array_equal(q2.codes, base.codes) and q2.n_out == base.n_out


def test_degenerate_inputs():
    z = np.zeros(33, np.float32)
    q = ref.quantize_grad(z, 1.0, 0.0, 4, rounding=1)
    assert q.c == 0 and q.scale == 0 and q.n_out == 0 and not q.codes.any()
    g = _grad(100)
    q = ref.quantize_grad(g, 1.0, 1.0, 4, n_nonfinite=1)
    assert not q.codes.any() and q.n_out == 0
    one = ref.quantize_grad(np.array([-2.5], np.float32), 1.0, 2.5, 4)
    assert list(one.codes) == [-7] and one.n_out == 0


# ------------------------------------------------------------------ quantizer, stochastic rounding
def test_sr_brackets_and_determinism():
    g = _grad(1 << 14, seed=5)
    gm, _ = ref.grad_stats(g)
    gamma, bits = 0.5, 4
    a = ref.quantize_grad(g, gamma, gm, bits, 1, seed=1, it=0)
    b = ref.quantize_grad(g, gamma, gm, bits, 1, seed=1, it=0)
    c = ref.quantize_grad(g, gamma, gm, bits, 1, seed=1, it=1)
    d = ref.quantize_grad(g, gamma, gm, bits, 1, seed=2, it=0)
    assert np.array_equal(a.codes, b.codes)
    assert not np.array_equal(a.codes, c.codes) and not np.array_equal(a.codes, d.codes)
    x = np.clip(g.astype(np.float64) / float(a.scale), -7, 7)
    fl = np.floor(np.float32(g) / a.scale).clip(-7, 7)
    assert np.all((a.codes == fl) | (a.codes == fl + 1))
    assert np.abs(x - a.codes).max() < 1.0 + 1e-6
    # clipped values and exact grid points are deterministic
    clipped = np.abs(g) > a.c
    assert np.all(np.abs(a.codes[clipped]) == 7) and np.array_equal(a.codes[clipped], c.codes[clipped])
    assert a.n_out == int(clipped.sum())


def test_sr_is_unbiased():
    """E[s q] = g for unclipped g: the mean over many element indices is within 4 sigma."""
    n = 1 << 18
    for frac in (0.125, 0.3, 0.77):
        val = np.float32((2 + frac) * 2.0 ** -8)
        g = np.full(n, val, np.float32)
        g[0] = np.float32(7 * 2.0 ** -8)             # fixes g_max so that s = 2^-8
        q = ref.quantize_grad(g, 1.0, g[0], 4, 1, seed=42, it=3)
        up = (q.codes[1:] == 3).mean()
        assert set(np.unique(q.codes[1:])) <= {2, 3}
        p = np.floor(frac * 65536) / 65536
        assert abs(up - p) < 4 * np.sqrt(p * (1 - p) / (n - 1))


def test_sr_threshold_uses_the_elements_own_random_field():
    """q = floor(x) + (u < t) with u the 16-bit field of the element's own index."""
    val = np.float32(2.5 * 2.0 ** -8)
    n = 64
    g = np.full(n, val, np.float32)
    g[0] = np.float32(7 * 2.0 ** -8)
    q = ref.quantize_grad(g, 1.0, g[0], 4, 1, seed=77, it=5)
    for i in range(1, n):
        assert q.codes[i] == 2 + (ref.rand16(77, 5, i) < 32768)


# ------------------------------------------------------------------ packing
def test_pack_layout():
    codes = np.array([1, -1, 7, -7, 0, 3, -8], np.int8)
    assert list(ref.pack(codes, 4)) == [0xF1, 0x97, 0x30, 0x08]
    assert list(ref.unpack4(ref.pack(codes, 4), 7, True)) == list(codes)
    assert list(ref.unpack4(np.array([0xF1], np.uint8), 2, False)) == [1, 15]
    assert ref.pack(codes, 6).view(np.int8).tolist() == codes.tolist()


# ------------------------------------------------------------------ ULG (Eq. 7 vs Eq. 8)
@pytest.mark.parametrize("bits", [4, 6, 8])
@pytest.mark.parametrize("gamma", [0.3, 0.6, 0.9, 1.0])
def test_error_of_large_gradients_is_below_ulg(bits, gamma):
    g = _grad(1 << 16, seed=21)
    gm, _ = ref.grad_stats(g)
    q = ref.quantize_grad(g, gamma, gm, bits)
    rep = analysis.large_gradient_report(g, ref.dequantize(q.codes, q.scale), 1e-3, gamma, bits)
    assert rep.n_in + rep.n_out == rep.n_large                      # Eq. (10)
    assert rep.e_large <= rep.u_large * (1 + 1e-5)                  # E(G_L) <= U(G_L)
    assert rep.n_out == min(q.n_out, rep.n_large)
    # stochastic rounding at most doubles the clip-in bound
    qs = ref.quantize_grad(g, gamma, gm, bits, 1, seed=1)
    reps = analysis.large_gradient_report(g, ref.dequantize(qs.codes, qs.scale), 1e-3, gamma, bits)
    u_in_part = (gamma / (2 ** bits - 2)) * reps.r_in / 1e-3
    assert reps.e_large_in <= 2 * u_in_part * (1 + 1e-5) + 1e-12


def test_sr_threshold_uses_the_exact_fractional_part():
    """t = trunc(frac(x) 2^16) with frac(x) = x - floor(x) exactly.  For x = -(1258 + 2^-10) / 2^16
    the exact threshold is 65536 - 1259 = 64277, while a binary32 subtraction x - floor(x) would
    round up to 64278 / 65536; the element whose random field is u = 64277 tells them apart."""
    seed, it = 5, 0
    i = next(k for k in range(1, 2_000_000) if ref.rand16(seed, it, k) == 64277)
    x = -(1258 + 2.0 ** -10) / 65536
    assert float(np.float32(x)) == x                       # representable
    g = np.zeros(i + 1, np.float32)
    g[0] = np.float32(7 * 2.0 ** -8)                       # g_max, so that s = 2^-8 and g / s is exact
    g[i] = np.float32(x * 2.0 ** -8)
    q = ref.quantize_grad(g, 1.0, g[0], 4, 1, seed, it)
    assert q.scale == np.float32(2.0 ** -8)
    assert q.codes[i] == -1                                # u < t is false: stays at floor(x)
    j = next(k for k in range(1, 2_000_000) if ref.rand16(seed, it, k) == 64276)
    g2 = np.zeros(j + 1, np.float32)
    g2[0], g2[j] = g[0], g[i]
    assert ref.quantize_grad(g2, 1.0, g2[0], 4, 1, seed, it).codes[j] == 0


def test_sr_threshold_of_a_vanishing_negative_quotient_is_65535():
    """frac(x) = x - floor(x) < 1 for every x, so t = trunc(frac 2^16) <= 65535 and the element whose
    random field is u = 65535 stays at floor(x) = -1 however close to zero the negative x is (down to
    values where 1 - |x| is no longer representable in binary64); every other u rounds it up to 0."""
    seed, it = 11, 3
    i = next(k for k in range(1, 2_000_000) if ref.rand16(seed, it, k) == 65535)
    j = next(k for k in range(1, 2_000_000) if ref.rand16(seed, it, k) == 65534)
    for tiny in (2.0 ** -20, 2.0 ** -40, 2.0 ** -60, 2.0 ** -100):
        g = np.zeros(max(i, j) + 1, np.float32)
        g[0] = np.float32(7 * 2.0 ** -8)                   # g_max: s = 2^-8, g / s exact
        g[i] = g[j] = np.float32(-tiny * 2.0 ** -8)
        q = ref.quantize_grad(g, 1.0, g[0], 4, 1, seed, it)
        assert q.codes[i] == -1 and q.codes[j] == 0
        g[i] = g[j] = np.float32(tiny * 2.0 ** -8)         # the positive twin never rounds up
        q = ref.quantize_grad(g, 1.0, g[0], 4, 1, seed, it)
        assert q.codes[i] == 0 and q.codes[j] == 0
