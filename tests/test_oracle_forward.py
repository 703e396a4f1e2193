"""Pins for the oracle's forward side (CPU only): the weight and activation quantizers of
Eq. (1)-(4) against closed forms, the error bounds of a uniform quantizer, symmetries and the
already pinned gradient quantizer; the integer forward product against library routines."""
import numpy as np
import pytest
import torch

from oracle import ref

BITS = [2, 3, 4, 6, 8]


def _laplace(n, scale, seed):
    return np.random.default_rng(seed).laplace(0.0, scale, n).astype(np.float32)


# ---------------------------------------------------------------------------- weights, Eq. (2)
@pytest.mark.parametrize("bits", BITS)
def test_weight_grid_points_map_to_their_code(bits):
    qmax = 2 ** (bits - 1) - 1
    c = np.float32(qmax * 2.0 ** -5)                     # s = 2^-5 exactly
    k = np.arange(-qmax, qmax + 1)
    codes, s = ref.quantize_weight((k * 2.0 ** -5).astype(np.float32), c, bits)
    assert s == np.float32(2.0 ** -5)
    assert np.array_equal(codes, k)


@pytest.mark.parametrize("bits", BITS)
def test_weight_codes_range_clipping_and_error_bounds(bits):
    qmax = 2 ** (bits - 1) - 1
    w = _laplace(200_000, 0.05, bits)
    c = np.float32(0.12)
    codes, s = ref.quantize_weight(w, c, bits)
    assert s == np.float32(c / np.float32(qmax))          # Eq. (2): one binary32 division
    assert codes.min() >= -qmax and codes.max() <= qmax   # 2^b - 1 levels, symmetric
    w64, q64 = w.astype(np.float64), float(s) * codes.astype(np.float64)
    inside = np.abs(w64) <= float(c)
    # inside the interval: at most half a step (plus the binary32 rounding of s and of the quotient)
    assert np.all(np.abs(w64 - q64)[inside] <= 0.5 * float(s) * (1 + 2.0 ** -12))
    # outside: the code saturates with the sign of the weight
    assert np.array_equal(codes[~inside], (np.sign(w[~inside]) * qmax).astype(np.int8))
    assert (~inside).any() and inside.any()


def test_weight_two_bits_is_ternary_and_ties_go_to_even():
    codes, s = ref.quantize_weight(np.array([-3, -0.6, -0.5, -0.4, 0, 0.4, 0.5, 0.6, 3], np.float32), 1.0, 2)
    assert s == np.float32(1.0)
    assert codes.tolist() == [-1, -1, 0, 0, 0, 0, 0, 1, 1]
    # s = 2^-3: halves of a step are exact, so these are true ties
    codes, s = ref.quantize_weight((np.array([0.5, 1.5, 2.5, 3.5, -0.5, -1.5, -2.5]) * 0.125).astype(np.float32),
                                   np.float32(7 * 0.125), 4)
    assert codes.tolist() == [0, 2, 2, 4, 0, -2, -2]


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_weight_quantizer_is_odd_monotone_and_scale_invariant(bits):
    w = _laplace(50_000, 0.05, 10 + bits)
    c = np.float32(0.1)
    codes, s = ref.quantize_weight(w, c, bits)
    neg, _ = ref.quantize_weight(-w, c, bits)
    assert np.array_equal(neg, -codes)
    order = np.argsort(w, kind="stable")
    assert np.all(np.diff(codes[order].astype(np.int32)) >= 0)
    for k in (-7, 5):
        scaled, s2 = ref.quantize_weight(w * np.float32(2.0 ** k), c * np.float32(2.0 ** k), bits)
        assert np.array_equal(scaled, codes) and s2 == s * np.float32(2.0 ** k)


@pytest.mark.parametrize("bits", [3, 4, 8])
def test_weight_quantizer_agrees_with_the_pinned_gradient_quantizer(bits):
    """With c_g = c (gamma = 1, g_max = c) and nearest rounding the gradient quantizer of Eq. (1), (2), (4)
    is the same map; it divides before it clips, the weight quantizer clips before it divides."""
    w = _laplace(100_000, 0.05, 20 + bits)
    c = np.float32(0.09)
    codes, s = ref.quantize_weight(w, c, bits)
    g = ref.quantize_grad(w, 1.0, c, bits, rounding=0)
    assert np.array_equal(codes, g.codes) and s == g.scale


def test_degenerate_clipping_values_give_zero_codes_and_zero_scale():
    w = _laplace(64, 1.0, 3)
    for c in (0.0, -1.0, float("nan"), float("inf")):
        codes, s = ref.quantize_weight(w, c, 4)
        assert not codes.any() and s == 0.0
        codes, s = ref.quantize_act(np.abs(w), c, 4)
        assert not codes.any() and s == 0.0


# ------------------------------------------------------------------------ activations, Eq. (3)
@pytest.mark.parametrize("bits", BITS)
def test_activation_grid_points_map_to_their_code(bits):
    levels = 2 ** bits - 1
    c = np.float32(levels * 2.0 ** -4)                   # s = 2^-4 exactly
    k = np.arange(0, levels + 1)
    codes, s = ref.quantize_act((k * 2.0 ** -4).astype(np.float32), c, bits)
    assert s == np.float32(2.0 ** -4)
    assert np.array_equal(codes, k)


@pytest.mark.parametrize("bits", BITS)
def test_activation_codes_range_clipping_and_error_bounds(bits):
    levels = 2 ** bits - 1
    x = np.maximum(_laplace(200_000, 0.5, 30 + bits), np.float32(-0.3))   # mostly "after a ReLU", some negatives
    c = np.float32(1.3)
    codes, s = ref.quantize_act(x, c, bits)
    assert s == np.float32(c / np.float32(levels))        # Eq. (3): 2^b - 1 steps on [0, c]
    assert codes.dtype == np.uint8 and codes.max() <= levels
    x64, q64 = x.astype(np.float64), float(s) * codes.astype(np.float64)
    inside = (x64 >= 0) & (x64 <= float(c))
    assert np.all(np.abs(x64 - q64)[inside] <= 0.5 * float(s) * (1 + 2.0 ** -12))
    assert not codes[x < 0].any()                         # clip(x, c) = min(max(x, 0), c)
    assert np.all(codes[x > c] == levels)
    assert (x < 0).any() and (x > c).any()
    order = np.argsort(x, kind="stable")
    assert np.all(np.diff(codes[order].astype(np.int32)) >= 0)


def test_activation_and_weight_quantizers_differ_as_eq_2_and_3_say():
    """Same input, same c, b = 4: 15 steps on [0, c] against 7 steps on each side of 0."""
    x = np.array([0.0, 0.25, 0.55, 1.0, -0.6], np.float32)
    a, sa = ref.quantize_act(x, 1.0, 4)
    w, sw = ref.quantize_weight(x, 1.0, 4)
    assert sa == np.float32(1.0) / np.float32(15) and sw == np.float32(1.0) / np.float32(7)
    assert a.tolist() == [0, 4, 8, 15, 0]                 # 3.75 -> 4, 8.25 -> 8, negative -> 0
    assert w.tolist() == [0, 2, 4, 7, -4]                 # 1.75 -> 2, 3.85 -> 4, -4.2 -> -4


# ------------------------------------------------------------------------ forward product
SHAPES = [
    ref.ConvShape(N=2, C=3, H=5, W=5, K=4, R=3, S=3, stride=1, pad=1),
    ref.ConvShape(N=2, C=2, H=6, W=6, K=3, R=3, S=3, stride=2, pad=1),
    ref.ConvShape(N=1, C=3, H=9, W=9, K=2, R=7, S=7, stride=2, pad=3),
    ref.ConvShape(N=3, C=4, H=4, W=6, K=5, R=1, S=1, stride=1, pad=0),
    ref.ConvShape(N=2, C=4, H=6, W=6, K=3, R=1, S=1, stride=2, pad=0),
    ref.ConvShape(N=1, C=2, H=5, W=7, K=2, R=3, S=3, stride=1, pad=0),
    ref.ConvShape(N=1, C=1, H=6, W=5, K=1, R=2, S=3, stride=2, pad=1),
]


def _codes(d, seed):
    rng = np.random.default_rng(seed)
    qW = rng.integers(-8, 8, (d.K, d.R, d.S, d.C)).astype(np.int16)
    qX = rng.integers(0, 16, (d.N, d.H, d.W, d.C)).astype(np.int16)
    qdY = rng.integers(-7, 8, (d.N, d.P, d.Q, d.K)).astype(np.int16)
    return qX, qW, qdY


@pytest.mark.parametrize("d", SHAPES, ids=lambda d: f"{d.R}x{d.S}s{d.stride}p{d.pad}")
def test_conv_forward_matches_library_convolution(d):
    qX, qW, _ = _codes(d, 1)
    y = torch.nn.functional.conv2d(torch.tensor(qX.transpose(0, 3, 1, 2).astype(np.float64)),
                                   torch.tensor(qW.transpose(0, 3, 1, 2).astype(np.float64)),
                                   stride=d.stride, padding=d.pad).numpy().transpose(0, 2, 3, 1)
    assert np.array_equal(ref.conv_forward(d, qX, qW), np.rint(y).astype(np.int64))


@pytest.mark.parametrize("d", SHAPES[:3], ids=lambda d: f"{d.R}x{d.S}s{d.stride}p{d.pad}")
def test_forward_is_the_adjoint_of_both_backward_contractions(d):
    """<dY, conv(X, W)> = <dgrad(dY, W), X> = <wgrad(dY, X), W>, all three from the oracle, in integers."""
    qX, qW, qdY = _codes(d, 2)
    lhs = int((qdY.astype(np.int64) * ref.conv_forward(d, qX, qW)).sum())
    assert lhs == int((ref.conv_backward("dgrad", d, qdY, qW) * qX).sum())
    assert lhs == int((ref.conv_backward("wgrad", d, qdY, qX) * qW).sum())


def test_linear_forward_matches_library_matmul_and_pointwise_conv():
    rng = np.random.default_rng(5)
    M, O, I = 13, 7, 21
    qX = rng.integers(0, 256, (M, I)).astype(np.int16)
    qW = rng.integers(-128, 128, (O, I)).astype(np.int16)
    want = qX.astype(np.int64) @ qW.astype(np.int64).T
    assert np.array_equal(ref.gemm_forward(qX, qW, M, O, I), want)
    d = ref.ConvShape(N=M, C=I, H=1, W=1, K=O, R=1, S=1)
    assert np.array_equal(ref.conv_forward(d, qX, qW).reshape(M, O), want)


def test_all_ones_forward_counts_the_taps_inside_the_image():
    d = ref.ConvShape(N=1, C=2, H=5, W=5, K=1, R=3, S=3, stride=1, pad=1)
    y = ref.conv_forward(d, np.ones((1, 5, 5, 2), np.int16), np.ones((1, 3, 3, 2), np.int16))[0, :, :, 0]
    rows = np.array([2, 3, 3, 3, 2])
    assert np.array_equal(y, 2 * np.outer(rows, rows))


def test_sampled_forward_outputs_and_threads_agree_with_full():
    d = SHAPES[1]
    qX, qW, _ = _codes(d, 7)
    full = ref.conv_forward(d, qX, qW)
    idx = np.random.default_rng(0).integers(0, full.size, 40)
    assert np.array_equal(ref.conv_forward(d, qX, qW, idx=idx), full.ravel()[idx])
    assert np.array_equal(ref.conv_forward(d, qX, qW, threads=3), full)
    M, O, I = 9, 5, 11
    a = np.random.default_rng(1).integers(0, 16, (M, I)).astype(np.int16)
    b = np.random.default_rng(2).integers(-8, 8, (O, I)).astype(np.int16)
    g = ref.gemm_forward(a, b, M, O, I)
    assert np.array_equal(ref.gemm_forward(a, b, M, O, I, idx=np.arange(M * O)[::3]), g.ravel()[::3])
    assert np.array_equal(ref.gemm_forward(a, b, M, O, I, threads=4), g)
