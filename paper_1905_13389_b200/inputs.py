"""Seeded synthetic inputs shared by the CUDA path's callers and the CPU oracle's callers.

This module holds no arithmetic of the method: it only draws float tensors with
the shapes and value distributions of the five workloads (stand-ins for the
ImageNet-style layers of the paper's Section 5 experiments, whose datasets and
trained weights are not available).  Everything is numpy on the host; the seed
of tensor ``t`` of workload ``c`` is ``190513389 + 1000*c + t``.
"""
from __future__ import annotations

import math

import numpy as np

BASE_SEED = 190513389

# (weight bits, activation bits) of the square-GEMM sweep
SWEEP_BITS = [(1, 1), (1, 2), (2, 2), (2, 3), (3, 3), (4, 4), (8, 8)]


def _rng(config: int, tensor: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(BASE_SEED + 1000 * config + tensor))


def normal(config: int, tensor: int, shape, std: float = 1.0, relu: bool = False) -> np.ndarray:
    """N(0, std^2) float32 tensor, optionally passed through ReLU."""
    x = _rng(config, tensor).standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    if relu:
        np.maximum(x, 0, out=x)
    return x


def uniform_levels(config: int, tensor: int, shape, bits: int) -> np.ndarray:
    """Floats in [-1, 1] that land uniformly on all 2^bits levels (range 1): the level centres
    (2u - L)/L.  Gaussian data under a max-abs range sits almost entirely on the two central
    levels, so parity cases add these to exercise every bit-plane."""
    L = (1 << bits) - 1
    u = _rng(config, tensor).integers(0, L + 1, size=shape)
    return ((2 * u - L) / np.float64(L)).astype(np.float32)


def config1():
    """Single GEMM, W2A2, m = n = 64, k = 512; per-tensor ranges."""
    return dict(name="gemm_w2a2_64x64x512", a_bits=2, w_bits=2, m=64, n=64, k=512,
                x=normal(1, 0, (64, 512), relu=True), w=normal(1, 1, (64, 512)), w_per_row=False)


def config2(batch: int = 64, n: int = 4096, k: int = 9216):
    """Fully-connected layer, W2A2: weights n x k N(0, 0.01^2) with a per-output-channel range,
    activations batch x k ReLU(N(0,1)) with a per-tensor range."""
    return dict(name="fc_w2a2_%dx%dx%d" % (batch, n, k), a_bits=2, w_bits=2, m=batch, n=n, k=k,
                x=normal(2, 0, (batch, k), relu=True), w=normal(2, 1, (n, k), std=0.01), w_per_row=True)


def config3(N: int = 32, C: int = 256, H: int = 14, W: int = 14, O: int = 256):
    """3x3 convolution, W3A3, stride 1, pad 1; Kaiming-normal weights (std = sqrt(2 / fan_in))."""
    return dict(name="conv3x3_w3a3_%dx%dx%dx%d" % (N, C, H, W), a_bits=3, w_bits=3, stride=1, pad=1,
                x=normal(3, 0, (N, C, H, W), relu=True),
                w=normal(3, 1, (O, C, 3, 3), std=math.sqrt(2.0 / (C * 9))))


def config4(w_bits: int, a_bits: int, size: int = 4096):
    """Square GEMM of the bit-width sweep: A = ReLU(N(0,1)) activations, B = N(0,1) weights."""
    return dict(name="gemm_w%da%d_%d" % (w_bits, a_bits, size), a_bits=a_bits, w_bits=w_bits,
                m=size, n=size, k=size,
                x=normal(4, 0, (size, size), relu=True), w=normal(4, 1, (size, size)), w_per_row=False)


# ResNet-18's quantized convolutions: (name, C_in, C_out, kernel, stride, input H = W)
RESNET18_QUANT_LAYERS = [
    ("layer1.0.conv1", 64, 64, 3, 1, 56), ("layer1.0.conv2", 64, 64, 3, 1, 56),
    ("layer1.1.conv1", 64, 64, 3, 1, 56), ("layer1.1.conv2", 64, 64, 3, 1, 56),
    ("layer2.0.conv1", 64, 128, 3, 2, 56), ("layer2.0.conv2", 128, 128, 3, 1, 28),
    ("layer2.0.downsample", 64, 128, 1, 2, 56),
    ("layer2.1.conv1", 128, 128, 3, 1, 28), ("layer2.1.conv2", 128, 128, 3, 1, 28),
    ("layer3.0.conv1", 128, 256, 3, 2, 28), ("layer3.0.conv2", 256, 256, 3, 1, 14),
    ("layer3.0.downsample", 128, 256, 1, 2, 28),
    ("layer3.1.conv1", 256, 256, 3, 1, 14), ("layer3.1.conv2", 256, 256, 3, 1, 14),
    ("layer4.0.conv1", 256, 512, 3, 2, 14), ("layer4.0.conv2", 512, 512, 3, 1, 7),
    ("layer4.0.downsample", 256, 512, 1, 2, 14),
    ("layer4.1.conv1", 512, 512, 3, 1, 7), ("layer4.1.conv2", 512, 512, 3, 1, 7),
]


def config5_weights():
    """Kaiming-normal weights of the 19 quantized convolutions plus the fp32 7x7 stem."""
    ws = {"conv1": normal(5, 1, (64, 3, 7, 7), std=math.sqrt(2.0 / (3 * 49)))}
    for t, (name, cin, cout, ksz, _, _) in enumerate(RESNET18_QUANT_LAYERS):
        ws[name] = normal(5, 10 + t, (cout, cin, ksz, ksz), std=math.sqrt(2.0 / (cin * ksz * ksz)))
    return ws


def config5_input(batch: int = 128, size: int = 224):
    """N(0,1) image batch, NCHW."""
    return normal(5, 0, (batch, 3, size, size))
