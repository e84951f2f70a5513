"""Pins of the oracle's full-precision glue (the test network's 7x7 stem and 3x3 max-pool, which are
not part of the paper's method): against float64 library convolution / pooling and closed forms."""
import numpy as np
import torch

import oracle
from paper_1905_13389_b200 import inputs


def test_stem_against_float64_convolution():
    x = inputs.config5_input(2, 37)                                   # odd size: ragged border on both sides
    w = inputs.config5_weights()["conv1"]
    y = oracle.stem(x, w, relu=False)
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double(), stride=2, padding=3).numpy()
    assert y.shape == ref.shape == (2, 64, 19, 19)
    assert np.abs(y - ref).max() <= 1e-5 * np.abs(ref).max()         # 147-term fp32 chains against float64
    assert np.array_equal(oracle.stem(x, w, relu=True), np.maximum(y, 0))


def test_stem_closed_forms():
    # a filter that is 1 at its centre tap of channel 1 only: output o = input channel 1 sampled at stride 2
    x = inputs.config5_input(1, 20)
    w = np.zeros((64, 3, 7, 7), np.float32)
    w[5, 1, 3, 3] = 1.0
    w[9, 2, 0, 6] = -2.0                                              # top-right tap: shifted, zero-padded view
    y = oracle.stem(x, w, relu=False)
    assert np.array_equal(y[0, 5], x[0, 1, ::2, ::2])
    shifted = np.zeros((10, 10), np.float32)
    for oh in range(10):
        for ow in range(10):
            ih, iw = 2 * oh - 3, 2 * ow + 3
            if 0 <= ih < 20 and 0 <= iw < 20:
                shifted[oh, ow] = -2.0 * x[0, 2, ih, iw]
    assert np.array_equal(y[0, 9], shifted)
    assert not y[0, 0].any()
    # all-ones input and filter: the count of in-image taps times 3 channels
    y = oracle.stem(np.ones((1, 3, 9, 9), np.float32), np.ones((64, 3, 7, 7), np.float32), relu=False)
    assert y[0, 0, 0, 0] == 3 * 4 * 4 and y[0, 63, 2, 2] == 3 * 7 * 7


def test_maxpool_against_library_and_padding():
    x = np.random.default_rng(0).standard_normal((2, 3, 11, 8)).astype(np.float32)
    ref = torch.nn.functional.max_pool2d(torch.from_numpy(x), 3, 2, 1).numpy()
    assert np.array_equal(oracle.maxpool3x3s2(x), ref)
    neg = -np.ones((1, 1, 4, 4), np.float32)                          # padding never wins, even over negatives
    assert np.array_equal(oracle.maxpool3x3s2(neg), -np.ones((1, 1, 2, 2), np.float32))
