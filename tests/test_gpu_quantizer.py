"""GPU parity: statistics, quantizer and interval update versus the CPU oracle, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2407_12637_b200 import lbt, synth

pytestmark = pytest.mark.gpu


def _run_gpu(g_host, bits, rounding, gamma=1.0, seed=0, it=0, alpha=1e-3, beta=1e-3, update=True):
    dY = torch.from_numpy(np.ascontiguousarray(g_host)).cuda()
    n = dY.numel()
    st = lbt.new_state(gamma=gamma, alpha=alpha, beta=beta, bits=bits, rounding=rounding, seed=seed, it=it)
    stats = lbt.new_stats()
    q = torch.full(((n + 1) // 2 if bits <= 4 else n,), 0xAB, dtype=torch.uint8, device="cuda")
    q = torch.cat([q, torch.full((64,), 0xCD, dtype=torch.uint8, device="cuda")])  # canary
    lbt.grad_stats(dY, st, stats)
    lbt.quantize_grad(dY, st, stats, q)
    if update:
        lbt.update_interval(st, stats)
    torch.cuda.synchronize()
    assert bool((q[-64:] == 0xCD).all()), "quantizer wrote past its output"
    return q[:-64].cpu().numpy(), lbt.read_stats(stats), lbt.read_state(st)


def _run_ref(g, bits, rounding, gamma=1.0, seed=0, it=0, alpha=1e-3, beta=1e-3):
    gm, bad = ref.grad_stats(g)
    q = ref.quantize_grad(g, gamma, gm, bits, rounding, seed, it, bad)
    new_gamma = ref.update_interval(gamma, alpha, beta, beta, 1.0, bits, g.size, q.n_out, bad)
    return ref.pack(q.codes, bits), gm, bad, q, new_gamma


def _compare(g, bits, rounding, **kw):
    packed_gpu, stats, st = _run_gpu(g, bits, rounding, **kw)
    packed_ref, gm, bad, q, new_gamma = _run_ref(g, bits, rounding, **kw)
    assert np.float32(stats.g_max) == gm
    assert stats.n == g.size and stats.n_nonfinite == bad
    assert np.float32(stats.c) == q.c and np.float32(stats.scale) == q.scale
    assert stats.n_out == q.n_out
    assert np.array_equal(packed_gpu, packed_ref)
    assert np.float32(st.gamma) == new_gamma
    assert st.iter == kw.get("it", 0) + 1
    return stats, st


@pytest.mark.parametrize("n", [1, 7, 8, 9, 15, 1000, 32768, (1 << 21) + 3])
@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("rounding", [0, 1])
def test_sizes_and_ragged_tails(n, bits, rounding):
    g = synth.laplace_outliers(n, 1e-3, seed=n)
    _compare(g, bits, rounding, gamma=0.73, seed=0x1234567890ABCDEF, it=(1 << 33) + 5)


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 7, 8])
def test_all_bit_widths(bits):
    g = synth.student_t3(100_003, 1e-4, seed=bits)
    for rounding in (0, 1):
        _compare(g, bits, rounding, gamma=0.41, seed=bits, it=3)


def test_config0_gradient():
    g = synth.laplace_outliers(128 * 256, 1e-3, seed=0)
    stats, st = _compare(g, 4, 1, seed=0)
    assert stats.n_out == 0 and np.float32(st.gamma) == np.float32(1.0) - np.float32(1e-3)


def test_degenerate_inputs():
    z = np.zeros(1000, np.float32)
    _compare(z, 4, 1)
    g = synth.laplace_outliers(5000, 1e-3, seed=1)
    g[[17, 4000]] = [np.inf, np.nan]
    packed, stats, st = _run_gpu(g, 4, 1, gamma=0.5)
    assert stats.n_nonfinite == 2 and not packed.any() and stats.n_out == 0
    assert st.dev_status == lbt.ERR_NONFINITE and np.float32(st.gamma) == np.float32(0.5)
    assert np.float32(stats.g_max) == ref.grad_stats(g)[0]


def test_empty_tensor():
    dY = torch.zeros(4, device="cuda")[:0]
    st, stats = lbt.new_state(), lbt.new_stats()
    lbt.lib().lbt_grad_stats(dY.data_ptr(), 0, st.data_ptr(), stats.data_ptr(), None, 0, 0)
    torch.cuda.synchronize()
    s = lbt.read_stats(stats)
    assert s.g_max == 0 and s.n == 0 and s.n_nonfinite == 0


def test_interval_trajectory_over_ten_drifting_steps():
    """ResNet-20-shaped layer (batch 128, 16 channels, 32x32): ten steps, scale x0.9 per step."""
    n = 128 * 32 * 32 * 16
    st = lbt.new_state(gamma=1.0, alpha=1e-3, beta=1e-3, bits=4, rounding=1, seed=7)
    stats = lbt.new_stats()
    q = torch.empty(n // 2, dtype=torch.uint8, device="cuda")
    gamma = np.float32(1.0)
    for t in range(10):
        g = synth.laplace_outliers(n, 1e-4 * 0.9 ** t, seed=7, stream=t)
        dY = torch.from_numpy(g).cuda()
        lbt.grad_stats(dY, st, stats)
        lbt.quantize_grad(dY, st, stats, q)
        lbt.update_interval(st, stats)
        torch.cuda.synchronize()
        gm, _ = ref.grad_stats(g)
        rq = ref.quantize_grad(g, gamma, gm, 4, 1, 7, t)
        assert np.array_equal(q.cpu().numpy(), ref.pack(rq.codes, 4))
        s = lbt.read_stats(stats)
        assert s.n_out == rq.n_out and np.float32(s.scale) == rq.scale
        gamma = ref.update_interval(gamma, 1e-3, 1e-3, 1e-3, 1.0, 4, n, rq.n_out)
        state = lbt.read_state(st)
        assert np.float32(state.gamma) == gamma and state.iter == t + 1


def test_bad_arguments_are_rejected_on_the_host():
    dY = torch.zeros(64, device="cuda")
    st, stats = lbt.new_state(), lbt.new_stats()
    L = lbt.lib()
    assert L.lbt_grad_stats(dY.data_ptr() + 4, 8, st.data_ptr(), stats.data_ptr(), None, 0, 0) == lbt.ERR_ALIGNMENT
    assert L.lbt_grad_stats(dY.data_ptr(), 8, st.data_ptr(), None, None, 0, 0) == lbt.ERR_INVALID_ARG
    assert L.lbt_quantize_grad(dY.data_ptr(), 8, None, stats.data_ptr(), dY.data_ptr(), None, 0, 0) == lbt.ERR_INVALID_ARG
    assert L.lbt_update_interval(None, stats.data_ptr(), 0) == lbt.ERR_INVALID_ARG


@pytest.mark.parametrize("scale", [1e-30, 1e-17, 1e-12, 1e-3, 1.0, 3e6, 1e19, 1e30])
def test_scales_across_the_exponent_range(scale):
    """Both the fast path (scale and gamma in its proven range) and the literal path must give the
    oracle's bits; dense value distributions make every code and many rounding ties occur."""
    rng = np.random.default_rng(int(abs(np.log10(scale)) * 7) + 1)
    n = 200_003
    g = (rng.standard_normal(n) * scale).astype(np.float32)
    g[:5000] = (rng.uniform(-1, 1, 5000) * scale * 4).astype(np.float32)
    g[5000:5400] = (rng.integers(-127, 128, 400) * np.float32(scale) * np.float32(2.0 ** -5)).astype(np.float32)
    g[5400:5500] = (rng.standard_normal(100) * scale * 1e-30).astype(np.float32)   # far below one step
    for bits, rounding, gamma in [(8, 1, 0.9), (8, 0, 0.37), (4, 1, 0.0009765625), (4, 1, 0.0005), (6, 1, 1.0), (2, 0, 0.5)]:
        _compare(g, bits, rounding, gamma=gamma, seed=99, it=4, beta=0.0)


def test_denormal_gradients():
    g = (np.random.default_rng(5).standard_normal(50_000) * 1e-41).astype(np.float32)
    _compare(g, 4, 1, gamma=0.8, seed=3)
    _compare(g, 8, 0, gamma=1.0, seed=3)


def test_vanishing_negative_quotients_at_the_top_random_field():
    """Negative gradients far below one step round up to 0 unless their random field is 65535 (the
    threshold trunc(frac 2^16) is 65535, never 65536); positive ones never round up."""
    seed, it = 11, 3
    top = [k for k in range(1, 400_000) if ref.rand16(seed, it, k) == 65535][:4]
    assert top
    n = top[-1] + 9
    g = np.zeros(n, np.float32)
    g[0] = np.float32(7 * 2.0 ** -8)
    for k, e in zip(top, (-20, -40, -60, -100)):
        g[k] = np.float32(-(2.0 ** e) * 2.0 ** -8)
        g[k + 1] = g[k]                                    # a neighbour with another random field
        g[k - 1] = -g[k]
    packed, stats, _ = _run_gpu(g, 4, 1, gamma=1.0, seed=seed, it=it)
    q = ref.quantize_grad(g, 1.0, g[0], 4, 1, seed, it)
    assert np.array_equal(packed, ref.pack(q.codes, 4))
    assert all(q.codes[k] == -1 for k in top)
