"""Pins for the oracle's integer backward contractions (CPU only): library gradients of a
library convolution / matmul, an im2col restatement, adjointness, closed-form tap counts."""
import numpy as np
import pytest
import torch

from oracle import ref

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
    qdY = rng.integers(-7, 8, (d.N, d.P, d.Q, d.K)).astype(np.int16)
    qW = rng.integers(-8, 8, (d.K, d.R, d.S, d.C)).astype(np.int16)
    qX = rng.integers(0, 16, (d.N, d.H, d.W, d.C)).astype(np.int16)
    return qdY, qW, qX


def _torch_grads(d, qdY, qW, qX):
    """dX, dW of a library convolution by automatic differentiation, binary64 (exact here)."""
    x = torch.tensor(qX.transpose(0, 3, 1, 2).astype(np.float64), requires_grad=True)
    w = torch.tensor(qW.transpose(0, 3, 1, 2).astype(np.float64), requires_grad=True)
    y = torch.nn.functional.conv2d(x, w, stride=d.stride, padding=d.pad)
    gy = torch.tensor(qdY.transpose(0, 3, 1, 2).astype(np.float64))
    assert y.shape == gy.shape
    y.backward(gy)
    dx = x.grad.numpy().transpose(0, 2, 3, 1)
    dw = w.grad.numpy().transpose(0, 2, 3, 1)
    return np.rint(dx).astype(np.int64), np.rint(dw).astype(np.int64), y.detach().numpy()


@pytest.mark.parametrize("d", SHAPES, ids=lambda d: f"{d.R}x{d.S}s{d.stride}p{d.pad}")
def test_conv_gradients_match_library_autograd(d):
    qdY, qW, qX = _codes(d, 1)
    dx, dw, _ = _torch_grads(d, qdY, qW, qX)
    assert np.array_equal(ref.conv_backward("dgrad", d, qdY, qW), dx)
    assert np.array_equal(ref.conv_backward("wgrad", d, qdY, qX), dw)


@pytest.mark.parametrize("d", SHAPES[:3], ids=lambda d: f"{d.R}x{d.S}s{d.stride}p{d.pad}")
def test_adjointness_exact_in_integers(d):
    """<dY, conv(X, W)> = <dgrad(dY, W), X> = <wgrad(dY, X), W>."""
    qdY, qW, qX = _codes(d, 2)
    _, _, y = _torch_grads(d, qdY, qW, qX)
    y = np.rint(y.transpose(0, 2, 3, 1)).astype(np.int64)
    lhs = int((qdY.astype(np.int64) * y).sum())
    assert lhs == int((ref.conv_backward("dgrad", d, qdY, qW) * qX).sum())
    assert lhs == int((ref.conv_backward("wgrad", d, qdY, qX) * qW).sum())


def _im2col(d, qX):
    cols = np.zeros((d.N, d.P, d.Q, d.R, d.S, d.C), np.int64)
    for n in range(d.N):
        for p in range(d.P):
            for q in range(d.Q):
                for r in range(d.R):
                    for s in range(d.S):
                        h, w = p * d.stride + r - d.pad, q * d.stride + s - d.pad
                        if 0 <= h < d.H and 0 <= w < d.W:
                            cols[n, p, q, r, s] = qX[n, h, w]
    return cols.reshape(d.N * d.P * d.Q, d.R * d.S * d.C)


@pytest.mark.parametrize("d", SHAPES[:3], ids=lambda d: f"{d.R}x{d.S}s{d.stride}p{d.pad}")
def test_wgrad_equals_gemm_on_explicit_im2col(d):
    qdY, _, qX = _codes(d, 3)
    cols = _im2col(d, qX)
    dw = qdY.reshape(-1, d.K).astype(np.int64).T @ cols
    assert np.array_equal(ref.conv_backward("wgrad", d, qdY, qX).reshape(d.K, -1), dw)


def test_pointwise_conv_is_the_linear_layer():
    d = SHAPES[3]
    qdY, qW, qX = _codes(d, 4)
    M = d.N * d.H * d.W
    a = ref.conv_backward("dgrad", d, qdY, qW).reshape(M, d.C)
    b = ref.gemm_backward("dgrad", qdY.reshape(M, d.K), qW.reshape(d.K, d.C), M, d.K, d.C)
    assert np.array_equal(a, b)
    a = ref.conv_backward("wgrad", d, qdY, qX).reshape(d.K, d.C)
    b = ref.gemm_backward("wgrad", qdY.reshape(M, d.K), qX.reshape(M, d.C), M, d.K, d.C)
    assert np.array_equal(a, b)


def test_linear_gradients_match_library_matmul():
    rng = np.random.default_rng(5)
    M, O, I = 7, 5, 6
    qdY = rng.integers(-127, 128, (M, O)).astype(np.int16)
    qW = rng.integers(-8, 8, (O, I)).astype(np.int16)
    qX = rng.integers(0, 256, (M, I)).astype(np.int16)
    assert np.array_equal(ref.gemm_backward("dgrad", qdY, qW, M, O, I),
                          qdY.astype(np.int64) @ qW.astype(np.int64))
    assert np.array_equal(ref.gemm_backward("wgrad", qdY, qX, M, O, I),
                          qdY.astype(np.int64).T @ qX.astype(np.int64))
    idx = np.array([0, 7, 29])
    assert np.array_equal(ref.gemm_backward("wgrad", qdY, qX, M, O, I, idx=idx),
                          (qdY.astype(np.int64).T @ qX.astype(np.int64)).ravel()[idx])
    full = ref.gemm_backward("dgrad", qdY, qW, M, O, I, threads=3)
    assert np.array_equal(full, qdY.astype(np.int64) @ qW.astype(np.int64))


def test_all_ones_give_tap_counts():
    """With every code equal to 1, dgrad counts the (k, r, s) taps that reach an input pixel and
    wgrad counts the output pixels a tap sees: interior 3x3/pad-1 pixels get 9K, corners 4K."""
    d = ref.ConvShape(N=2, C=2, H=6, W=6, K=3, R=3, S=3, stride=1, pad=1)
    one = lambda *s: np.ones(s, np.int16)
    dx = ref.conv_backward("dgrad", d, one(d.N, d.P, d.Q, d.K), one(d.K, 3, 3, d.C))
    assert dx[0, 2, 3, 0] == 9 * d.K and dx[1, 0, 0, 1] == 4 * d.K and dx[0, 0, 3, 0] == 6 * d.K
    dw = ref.conv_backward("wgrad", d, one(d.N, d.P, d.Q, d.K), one(d.N, d.H, d.W, d.C))
    assert dw[0, 1, 1, 0] == d.N * 36 and dw[2, 0, 0, 1] == d.N * 25 and dw[1, 0, 1, 0] == d.N * 30


def test_sampled_outputs_and_threads_agree_with_full():
    d = SHAPES[1]
    qdY, qW, qX = _codes(d, 6)
    full = ref.conv_backward("dgrad", d, qdY, qW)
    idx = np.array([0, 5, 17, full.size - 1])
    assert np.array_equal(ref.conv_backward("dgrad", d, qdY, qW, idx=idx), full.ravel()[idx])
    assert np.array_equal(ref.conv_backward("dgrad", d, qdY, qW, threads=4), full)
    fw = ref.conv_backward("wgrad", d, qdY, qX)
    assert np.array_equal(ref.conv_backward("wgrad", d, qdY, qX, idx=idx[:3]), fw.ravel()[idx[:3]])


def test_epilogue_scales_once_and_flags_overflow():
    acc = np.array([0, 1, -3, 2**31, 12345], np.int64)
    out, over = ref.epilogue(acc, 0.01, 0.05)
    s = np.float32(0.01) * np.float32(0.05)
    assert over == 1
    assert np.array_equal(out, acc.astype(np.float32) * s)
