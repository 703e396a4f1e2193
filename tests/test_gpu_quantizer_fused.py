"""GPU parity of the one-launch quantizer (statistics, grid barrier, quantizer, clipping-factor update in
one cooperative kernel) versus the CPU oracle, bit for bit, and versus the three separate calls."""
import numpy as np
import pytest
import torch

from paper_2407_12637_b200 import lbt, synth
from tests.test_gpu_quantizer import _run_gpu, _run_ref

pytestmark = pytest.mark.gpu


def _run_fused(g_host, bits, rounding, gamma=1.0, seed=0, it=0, alpha=1e-3, beta=1e-3):
    dY = torch.from_numpy(np.ascontiguousarray(g_host)).cuda()
    n = dY.numel()
    st = lbt.new_state(gamma=gamma, alpha=alpha, beta=beta, bits=bits, rounding=rounding, seed=seed, it=it)
    stats = torch.full((40,), 0x5A, dtype=torch.uint8, device="cuda")     # stale contents must not matter
    q = torch.full(((n + 1) // 2 if bits <= 4 else n,), 0xAB, dtype=torch.uint8, device="cuda")
    q = torch.cat([q, torch.full((64,), 0xCD, dtype=torch.uint8, device="cuda")])  # canary
    lbt.quantize_grad_fused(dY, st, stats, q)
    torch.cuda.synchronize()
    assert bool((q[-64:] == 0xCD).all()), "quantizer wrote past its output"
    return q[:-64].cpu().numpy(), lbt.read_stats(stats), lbt.read_state(st)


def _compare(g, bits, rounding, **kw):
    packed_gpu, stats, st = _run_fused(g, bits, rounding, **kw)
    packed_ref, gm, bad, q, new_gamma = _run_ref(g, bits, rounding, **kw)
    assert np.float32(stats.g_max) == gm
    assert stats.n == g.size and stats.n_nonfinite == bad and stats.reserved == 0
    assert np.float32(stats.c) == q.c and np.float32(stats.scale) == q.scale
    assert stats.n_out == q.n_out
    assert np.array_equal(packed_gpu, packed_ref)
    assert np.float32(st.gamma) == new_gamma
    assert st.iter == kw.get("it", 0) + 1 and st.dev_status == 0
    return stats, st


@pytest.mark.parametrize("n", [1, 7, 8, 9, 1000, 32768, (1 << 21) + 3, 12_845_056])
@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("rounding", [0, 1])
def test_sizes_and_ragged_tails(n, bits, rounding):
    g = synth.laplace_outliers(n, 1e-3, seed=n)
    _compare(g, bits, rounding, gamma=0.73, seed=0x1234567890ABCDEF, it=(1 << 33) + 5)


@pytest.mark.parametrize("n_extra", [-8, 0, 1, 8 * 256 + 3])
def test_cached_random_words_boundary(n_extra):
    """With stochastic rounding a thread generates the Philox words of its first nine groups during the
    abs-max phase and reads them back in the quantize phase; later groups are generated in place. Sizes
    on both sides of "exactly nine groups per thread" of a full grid (148 x 4 blocks of 256 threads)."""
    n = 9 * 8 * 148 * 4 * 256 + n_extra
    g = synth.laplace_outliers(n, 1e-3, seed=n)
    _compare(g, 4, 1, gamma=0.61, seed=0xFEDCBA9876543210, it=7)


@pytest.mark.parametrize("bits", [2, 3, 5, 6, 7])
def test_other_bit_widths(bits):
    g = synth.student_t3(100_003, 1e-4, seed=bits)
    for rounding in (0, 1):
        _compare(g, bits, rounding, gamma=0.41, seed=bits, it=3)


def test_degenerate_inputs():
    _compare(np.zeros(1000, np.float32), 4, 1)
    g = synth.laplace_outliers(5000, 1e-3, seed=1)
    g[[17, 4000]] = [np.inf, np.nan]
    packed, stats, st = _run_fused(g, 4, 1, gamma=0.5)
    assert stats.n_nonfinite == 2 and not packed.any() and stats.n_out == 0
    assert st.dev_status == lbt.ERR_NONFINITE and np.float32(st.gamma) == np.float32(0.5) and st.iter == 1


def test_trajectory_equals_the_three_separate_calls():
    """Ten iterations with carried state: the fused and the separate paths stay identical."""
    n = 300_000
    st_a = lbt.new_state(gamma=1.0, alpha=1e-3, beta=1e-2, bits=4, rounding=1, seed=7)
    st_b = st_a.clone()
    stats_a, stats_b = lbt.new_stats(), lbt.new_stats()
    q_a = torch.empty(n // 2, dtype=torch.uint8, device="cuda")
    q_b = torch.empty(n // 2, dtype=torch.uint8, device="cuda")
    for step in range(10):
        dY = torch.from_numpy(synth.laplace_outliers(n, 1e-3 * 0.9 ** step, seed=step)).cuda()
        lbt.quantize_grad_fused(dY, st_a, stats_a, q_a)
        lbt.grad_stats(dY, st_b, stats_b)
        lbt.quantize_grad(dY, st_b, stats_b, q_b)
        lbt.update_interval(st_b, stats_b)
        torch.cuda.synchronize()
        assert torch.equal(q_a, q_b) and torch.equal(st_a, st_b) and torch.equal(stats_a, stats_b)


def test_tensor_far_beyond_l2_still_matches():
    n = 80_000_003                                                        # 320 MB: correct at any size
    g = synth.laplace_outliers(n, 1e-3, seed=3)
    _compare(g, 4, 1, gamma=0.6, seed=11, it=2)
