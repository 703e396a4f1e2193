"""Layer shapes of the benchmark configurations (convolutions as N, C, H, W, K, R, S, stride, pad).

The architectures are the published ResNet-20 (CIFAR), ResNet-18 / ResNet-50 (ImageNet) and EDSR
layer shapes the paper trains (Sec. 4.1); the values flowing through them are synthetic.
"""
from __future__ import annotations


def conv(N, C, H, W, K, R, S, stride=1, pad=0):
    return dict(N=N, C=C, H=H, W=W, K=K, R=R, S=S, stride=stride, pad=pad)


def linear(M, O, I):
    """A linear layer dY[M,O], W[O,I], X[M,I] as the 1x1 convolution on a 1x1 image."""
    return conv(M, I, 1, 1, O, 1, 1)


def out_hw(s):
    p = (s["H"] + 2 * s["pad"] - s["R"]) // s["stride"] + 1
    q = (s["W"] + 2 * s["pad"] - s["S"]) // s["stride"] + 1
    return p, q


def macs(s) -> int:
    """Multiply-accumulates of one contraction (dgrad and wgrad each)."""
    p, q = out_hw(s)
    return s["N"] * p * q * s["K"] * s["R"] * s["S"] * s["C"]


def grad_elems(s) -> int:
    p, q = out_hw(s)
    return s["N"] * p * q * s["K"]


CONFIG0 = {"linear_128x256x256": linear(128, 256, 256)}

CONFIG1 = {"resnet20_3x3_16": conv(128, 16, 32, 32, 16, 3, 3, 1, 1)}

CONFIG2 = {
    "resnet50_1x1_1024_256": conv(256, 1024, 14, 14, 256, 1, 1),
    "resnet50_3x3_256_256": conv(256, 256, 14, 14, 256, 3, 3, 1, 1),
    "resnet50_1x1_256_1024": conv(256, 256, 14, 14, 1024, 1, 1),
}

# (shape, how many layers of ResNet-18 have it)
CONFIG3 = {
    "conv1": (conv(256, 3, 224, 224, 64, 7, 7, 2, 3), 1),
    "layer1": (conv(256, 64, 56, 56, 64, 3, 3, 1, 1), 4),
    "layer2.0.conv1": (conv(256, 64, 56, 56, 128, 3, 3, 2, 1), 1),
    "layer2": (conv(256, 128, 28, 28, 128, 3, 3, 1, 1), 3),
    "layer2.downsample": (conv(256, 64, 56, 56, 128, 1, 1, 2, 0), 1),
    "layer3.0.conv1": (conv(256, 128, 28, 28, 256, 3, 3, 2, 1), 1),
    "layer3": (conv(256, 256, 14, 14, 256, 3, 3, 1, 1), 3),
    "layer3.downsample": (conv(256, 128, 28, 28, 256, 1, 1, 2, 0), 1),
    "layer4.0.conv1": (conv(256, 256, 14, 14, 512, 3, 3, 2, 1), 1),
    "layer4": (conv(256, 512, 7, 7, 512, 3, 3, 1, 1), 3),
    "layer4.downsample": (conv(256, 256, 14, 14, 512, 1, 1, 2, 0), 1),
    "fc": (linear(256, 1000, 512), 1),
}

CONFIG4 = {
    "gemm_8192": linear(8192, 8192, 8192),
    "edsr_3x3_64": conv(16, 64, 96, 96, 64, 3, 3, 1, 1),
}
