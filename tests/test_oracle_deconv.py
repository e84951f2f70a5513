"""Pins for the oracle's deconvolution (transposed convolution), CPU only.

The oracle spreads every input pixel over its output window (the definition).  It is checked
against forms that share nothing with that loop: the gather form written out per output element,
the library's own transposed convolution in float64 (exact on these small integers), the identity
with an ordinary convolution of the zero-stuffed input by the flipped filter (the oracle's conv is
pinned on its own), the adjoint identity <deconv(x), y> = <x, conv(y)>, and closed forms.
"""
import numpy as np
import pytest
import torch

import oracle

CASES = [  # KH, KW, stride, pad
    (4, 4, 2, 1), (2, 2, 2, 0), (3, 3, 2, 1), (3, 3, 2, 0), (3, 3, 1, 1), (4, 4, 1, 0),
    (2, 3, 2, 1), (4, 2, 2, 0), (1, 1, 1, 0), (3, 4, 1, 2),
]


def _ints(rng, shape, L=7):
    return (2 * rng.integers(0, L + 1, shape) - L).astype(np.int16)        # odd integers, |q| <= L (Eq. 20)


def _gather_form(qx, qw, stride, pad):
    """y[n,o,oh,ow] = sum over (c,kh,kw) with (oh + pad - kh) divisible by the stride and the quotient inside the image."""
    N, C, H, W = qx.shape
    O, _, KH, KW = qw.shape
    Ho, Wo = (H - 1) * stride - 2 * pad + KH, (W - 1) * stride - 2 * pad + KW
    y = np.zeros((N, O, Ho, Wo), dtype=np.int64)
    for oh in range(Ho):
        for ow in range(Wo):
            for kh in range(KH):
                for kw in range(KW):
                    th, tw = oh + pad - kh, ow + pad - kw
                    if th % stride or tw % stride:
                        continue
                    ih, iw = th // stride, tw // stride
                    if 0 <= ih < H and 0 <= iw < W:
                        y[:, :, oh, ow] += qx[:, :, ih, iw].astype(np.int64) @ qw[:, :, kh, kw].astype(np.int64).T
    return y


@pytest.mark.parametrize("KH,KW,stride,pad", CASES)
def test_deconv_equals_gather_form_and_library(KH, KW, stride, pad):
    rng = np.random.default_rng(100 * KH + 10 * KW + stride + pad)
    N, C, H, W, O = 2, 5, 4, 3, 3
    if (H - 1) * stride - 2 * pad + KH <= 0 or (W - 1) * stride - 2 * pad + KW <= 0:
        pytest.skip("empty output")
    qx, qw = _ints(rng, (N, C, H, W)), _ints(rng, (O, C, KH, KW), 3)
    got = oracle.deconv(qx, qw, stride, pad)
    assert np.array_equal(got, _gather_form(qx, qw, stride, pad))
    # the library routine wants the filter input-channel first: [C][O][KH][KW]
    lib = torch.nn.functional.conv_transpose2d(torch.from_numpy(qx.astype(np.float64)),
                                               torch.from_numpy(qw.astype(np.float64)).transpose(0, 1).contiguous(),
                                               stride=stride, padding=pad)
    assert got.shape == tuple(lib.shape)
    assert np.array_equal(got.astype(np.float64), lib.numpy())


@pytest.mark.parametrize("KH,KW,stride,pad", [(4, 4, 2, 1), (3, 3, 2, 1), (2, 2, 2, 0), (3, 3, 1, 1)])
def test_deconv_is_conv_of_the_zero_stuffed_input_by_the_flipped_filter(KH, KW, stride, pad):
    rng = np.random.default_rng(7)
    N, C, H, W, O = 1, 4, 5, 4, 3
    qx, qw = _ints(rng, (N, C, H, W)), _ints(rng, (O, C, KH, KW), 3)
    stuffed = np.zeros((N, C, (H - 1) * stride + 1, (W - 1) * stride + 1), dtype=np.int16)
    stuffed[:, :, ::stride, ::stride] = qx
    ph, pw = KH - 1 - pad, KW - 1 - pad                          # full padding minus the deconvolution's
    padded = np.pad(stuffed, ((0, 0), (0, 0), (ph, ph), (pw, pw)))
    ref = oracle.conv(padded, qw[:, :, ::-1, ::-1], 1, 0)
    assert np.array_equal(oracle.deconv(qx, qw, stride, pad), ref)


@pytest.mark.parametrize("KH,KW,stride,pad", [(4, 4, 2, 1), (3, 3, 2, 0), (2, 2, 2, 0)])
def test_deconv_is_the_adjoint_of_conv(KH, KW, stride, pad):
    """<deconv_w(x), y> = <x, conv_w'(y)> with w' the same filter read [C][O] (input and output swapped)."""
    rng = np.random.default_rng(11)
    N, C, H, W, O = 2, 3, 4, 5, 4
    qx, qw = _ints(rng, (N, C, H, W)), _ints(rng, (O, C, KH, KW), 3)
    up = oracle.deconv(qx, qw, stride, pad)
    y = _ints(rng, up.shape, 5)
    down = oracle.conv(y, np.ascontiguousarray(qw.transpose(1, 0, 2, 3)), stride, pad)
    assert down.shape == qx.shape
    assert int((up.astype(np.int64) * y).sum()) == int((qx.astype(np.int64) * down).sum())


def test_deconv_closed_forms():
    # kernel = stride, no padding: every output is reached by exactly one tap of one pixel
    qx = np.full((1, 6, 3, 3), 3, np.int16)
    qw = np.full((2, 6, 2, 2), -1, np.int16)
    assert np.array_equal(oracle.deconv(qx, qw, 2, 0), np.full((1, 2, 6, 6), -18, np.int32))
    # 4 x 4, stride 2, pad 1: interior outputs see 2 x 2 taps, border rows / columns 1 x 2, corners 1 x 1
    qx = np.ones((1, 5, 4, 4), np.int16)
    qw = np.ones((1, 5, 4, 4), np.int16)
    y = oracle.deconv(qx, qw, 2, 1)[0, 0]
    assert y.shape == (8, 8)
    assert np.all(y[1:-1, 1:-1] == 20) and np.all(y[0, 1:-1] == 10) and np.all(y[1:-1, -1] == 10)
    assert y[0, 0] == y[0, -1] == y[-1, 0] == y[-1, -1] == 5
    # a single input pixel paints the (channel-summed) filter at its window, cropped by the padding
    qx = np.zeros((1, 2, 3, 3), np.int16); qx[0, :, 1, 2] = (1, -1)
    qw = _ints(np.random.default_rng(3), (2, 2, 3, 3), 3)
    y = oracle.deconv(qx, qw, 2, 1)
    painted = (qw[:, 0] - qw[:, 1]).astype(np.int32)              # [O][3][3]
    assert y.shape == (1, 2, 5, 5)
    assert np.array_equal(y[0, :, 1:4, 3:5], painted[:, :, :2])   # window starts at (1, 3); its last column is cropped
    y[0, :, 1:4, 3:5] = 0
    assert not y.any()


def test_deconv_overflow_is_reported():
    qx = np.full((1, 32768, 2, 2), 255, np.int16)
    qw = np.full((1, 32768, 2, 2), 255, np.int16)
    with pytest.raises(OverflowError):
        oracle.deconv(qx, qw, 1, 0)                              # the centre output sums 4 * 32768 * 255^2 > 2^31


@pytest.mark.parametrize("per_channel,act", [(True, oracle.HRELU), (False, oracle.HTANH)])
def test_deconv_layer_composes_the_steps(per_channel, act):
    rng = np.random.default_rng(5)
    x = rng.standard_normal((2, 6, 3, 4)).astype(np.float32)
    w = rng.standard_normal((4, 6, 4, 4)).astype(np.float32)
    acc, out, s_a, s_w = oracle.deconv_layer(x, w, 3, 2, 2, 1, per_channel, act)
    want_sa = np.float32(np.abs(x).max() if act == oracle.HTANH else x.max())
    assert s_a[0] == want_sa
    assert np.array_equal(s_w, np.abs(w).reshape(4, -1).max(axis=1) if per_channel else np.abs(w).max(keepdims=True).reshape(1))
    qx = oracle.quantize(x, s_a, 3, act=act)
    qw = oracle.quantize(w, s_w, 2, per_row=per_channel)
    assert np.array_equal(acc, _gather_form(qx, qw, 2, 1))
    alpha = (np.float32(s_a[0]) / np.float32(7)) * (s_w.astype(np.float32) / np.float32(3))
    alpha = np.broadcast_to(alpha, (4,)).reshape(1, 4, 1, 1)
    assert np.array_equal(out, acc.astype(np.float32) * alpha.astype(np.float32))
