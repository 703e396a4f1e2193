"""Pins for the oracle's sort-based error metrics of Sec. 3.2-3.3 (E(G), E(G_L), U(G_L), R_in, R_out):
a worked example done by hand, the tie rule, and identities the definitions imply."""
import numpy as np

from oracle import analysis, ref


def test_worked_example_by_hand():
    """N = 8, alpha = 3/8 -> G_L = {8, -7, 6}; gamma = 0.75 -> c = 6; b = 3 -> qmax = 3, s = 2.
    Q = {6, -6, 6, 4, -0, 0, 2, -4}: errors {2, 1, 0, 1, 1, 0.5, 0, 1}."""
    g = np.array([8, -7, 6, 5, -1, 0.5, 2, -3], np.float32)
    q = ref.quantize_grad(g, 0.75, 8.0, 3, rounding=0)
    assert q.codes.tolist() == [3, -3, 3, 2, 0, 0, 1, -2] and q.scale == 2.0 and q.c == 6.0 and q.n_out == 2
    rep = analysis.large_gradient_report(g, ref.dequantize(q.codes, q.scale), 0.375, 0.75, 3)
    assert (rep.n, rep.n_large, rep.n_in, rep.n_out) == (8, 3, 1, 2)
    assert rep.r_in == 1 / 8 and rep.r_out == 2 / 8                      # Eq. (9)
    assert rep.e_all == 6.5 / (8 * 8)                                    # Eq. (5)
    assert rep.e_large == 3.0 / (3 * 8)                                  # Eq. (6): (2 + 1 + 0) / (N(G_L) g_max)
    assert rep.e_large_in == 0.0 and rep.e_large_out == 0.125            # Eq. (7)
    want_u = ((0.75 / 6) * (1 / 8) + 0.25 * (2 / 8)) / (3 / 8)           # Eq. (8), 2^b - 2 = 6
    assert abs(rep.u_large - want_u) < 1e-15
    assert rep.e_large <= rep.u_large


def test_equal_magnitudes_enter_the_large_set_in_memory_order():
    g = np.array([1, 2, -2, 2, 0.5, 2], np.float32)
    qg = np.array([1, 2, -1, 0, 0.5, -3], np.float64)                    # errors 0, 0, 1, 2, 0, 5
    rep = analysis.large_gradient_report(g, qg, 2 / 6, 1.0, 4)           # N(G_L) = 2: the first two of the four 2s
    assert rep.n_large == 2 and rep.e_large == (0 + 1) / (2 * 2)
    rep = analysis.large_gradient_report(g, qg, 3 / 6, 1.0, 4)           # N(G_L) = 3: the third 2 joins
    assert rep.n_large == 3 and rep.e_large == (0 + 1 + 2) / (3 * 2)


def test_identities_of_the_definitions():
    g = np.random.default_rng(3).laplace(0, 1e-3, 50_000).astype(np.float32)
    gm, _ = ref.grad_stats(g)
    for gamma in (1.0, 0.6, 0.3):
        q = ref.quantize_grad(g, gamma, gm, 4, rounding=0)
        rep = analysis.large_gradient_report(g, ref.dequantize(q.codes, q.scale), 1e-2, gamma, 4, c=q.c)
        assert rep.n_large == 500 and rep.n_in + rep.n_out == rep.n_large                 # Eq. (10)
        assert abs(rep.r_in + rep.r_out - rep.n_large / rep.n) < 1e-15
        assert rep.n_out == min(q.n_out, rep.n_large)                                    # G_out = G_L beyond c
        assert abs(rep.e_large - (rep.e_large_in + rep.e_large_out)) < 1e-15              # Eq. (7)
        assert rep.e_large <= rep.u_large * (1 + 1e-6)                                    # Eq. (7) vs Eq. (8)
    # gamma = 1: nothing is clipped, the large gradients' error is rounding error only
    q = ref.quantize_grad(g, 1.0, gm, 4, rounding=0)
    rep = analysis.large_gradient_report(g, ref.dequantize(q.codes, q.scale), 1e-2, 1.0, 4, c=q.c)
    assert rep.n_out == 0 and rep.e_large_out == 0.0
