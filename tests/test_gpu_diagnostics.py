"""GPU parity of the Sec. 3.2-3.3 diagnostics (E(G), E(G_L), U(G_L), clip ratios) with the oracle's
sort-based definitions: counts and the threshold exactly, binary64 sums within 1e-12 relative."""
import numpy as np
import pytest
import torch

from oracle import analysis, ref
from paper_2407_12637_b200 import lbt, synth

pytestmark = pytest.mark.gpu


def _run(g, bits, rounding, gamma, alpha, seed=3):
    dY = torch.from_numpy(g).cuda()
    st = lbt.new_state(gamma=gamma, alpha=alpha, bits=bits, rounding=rounding, seed=seed)
    stats = lbt.new_stats()
    q = torch.empty((g.size + 1) // 2 if bits <= 4 else g.size, dtype=torch.uint8, device="cuda")
    lbt.grad_stats(dY, st, stats)
    lbt.quantize_grad(dY, st, stats, q)
    d = lbt.grad_diagnostics(dY, q, bits, alpha, stats)
    gm, _ = ref.grad_stats(g)
    qr = ref.quantize_grad(g, gamma, gm, bits, rounding, seed, 0)
    a32 = float(np.float32(alpha))
    rep = analysis.large_gradient_report(g, float(qr.scale) * qr.codes.astype(np.float64), a32,
                                         float(qr.c) / float(gm), bits, c=qr.c)
    return d, rep, qr


def _check(d, rep):
    assert (d.n, d.n_large, d.n_in, d.n_out) == (rep.n, rep.n_large, rep.n_in, rep.n_out)
    for got, want in ((d.e_all, rep.e_all), (d.e_large, rep.e_large), (d.u_large, rep.u_large)):
        assert abs(got - want) <= 1e-12 * abs(want) + 1e-300


@pytest.mark.parametrize("n", [1, 9, 1000, 300_003, 4_000_000])
@pytest.mark.parametrize("bits,rounding", [(4, 0), (4, 1), (8, 1)])
def test_diagnostics_match_the_sort_based_oracle(n, bits, rounding):
    g = synth.laplace_outliers(n, 1e-3, seed=n % 97)
    for gamma, alpha in ((1.0, 1e-2), (0.5, 1e-3), (0.2, 0.3)):
        d, rep, _ = _run(g, bits, rounding, gamma, alpha)
        _check(d, rep)


def test_threshold_and_ties_in_memory_order():
    """Many equal magnitudes at the threshold: the earlier ones belong to G_L (as the oracle's stable sort)."""
    rng = np.random.default_rng(5)
    g = rng.choice(np.array([0.25, -0.25, 0.5, -0.5, 1.0, 2.0, -2.0], np.float32), 100_000).astype(np.float32)
    g[::1000] = 3.0
    for alpha in (0.05, 0.2, 0.5, 1.0, 0.0):
        d, rep, _ = _run(g, 4, 1, 0.4, alpha)          # stochastic rounding: tied elements have different errors
        _check(d, rep)
        if rep.n_large:
            order = np.argsort(-np.abs(g), kind="stable")
            assert d.threshold == np.abs(g)[order[rep.n_large - 1]]


def test_worked_example():
    g = np.array([8, -7, 6, 5, -1, 0.5, 2, -3], np.float32)
    d, rep, qr = _run(g, 3, 0, 0.75, 0.375)
    assert (d.n_large, d.n_in, d.n_out) == (3, 1, 2) and d.threshold == 6.0
    assert d.e_all == 6.5 / 64 and d.e_large == 0.125 and d.sum_large_out == 3.0 and d.sum_large_in == 0.0
    assert abs(d.u_large - ((0.75 / 6) * (1 / 8) + 0.25 * (2 / 8)) / (3 / 8)) < 1e-15


def test_rejections():
    L = lbt.lib()
    buf = torch.zeros(4096, device="cuda")
    p = buf.data_ptr()
    need = L.lbt_diagnostics_workspace_bytes()
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    assert L.lbt_grad_diagnostics(p, 64, p, 4, 0.5, p, p, ws.data_ptr(), need - 1, 0) == lbt.ERR_WORKSPACE
    assert L.lbt_grad_diagnostics(p, 64, p, 9, 0.5, p, p, ws.data_ptr(), need, 0) == lbt.ERR_UNSUPPORTED_BITS
    assert L.lbt_grad_diagnostics(p, 0, p, 4, 0.5, p, p, ws.data_ptr(), need, 0) == lbt.ERR_INVALID_ARG
    assert L.lbt_grad_diagnostics(p, 64, p, 4, 1.5, p, p, ws.data_ptr(), need, 0) == lbt.ERR_INVALID_ARG
