"""Pins for the oracle's layer product, convolution and decoder scale (CPU only).

The integer product is checked against the M x K branch decomposition by brute
force over every code (Eq. 7-10), against the {0,1}-encoding polynomial of
Eq. 17, against the sign-binarised dot at 1 bit (Eq. 14), against closed forms,
and against numpy's own matmul / sliding-window einsum.  The scale is checked
against the "1/9" of Fig. 1 and Eq. 18 in exact rationals.
"""
import itertools
from fractions import Fraction

import numpy as np
import pytest

import oracle


def _planes(u: np.ndarray, bits: int):
    """Bit-planes of the level index: plane p holds bit p (weight 2^p) as 0/1 per element."""
    return [((u >> p) & 1) for p in range(bits)]


def _branch_sum(ua, ub, a_bits, w_bits):
    """Eq. 9 with the {-1,+1} elements of Eq. 10, each binary dot taken as n - 2*popcount(xor)."""
    n = len(ua)
    pa, pb = _planes(np.asarray(ua), a_bits), _planes(np.asarray(ub), w_bits)
    total = 0
    for i in range(a_bits):
        for j in range(w_bits):
            popc = int(np.count_nonzero(pa[i] ^ pb[j]))
            total += (1 << (i + j)) * (n - 2 * popc)
    return total


@pytest.mark.parametrize("a_bits,w_bits,n", [(1, 1, 4), (1, 2, 3), (2, 2, 3), (2, 3, 3), (3, 3, 2), (3, 1, 3), (4, 4, 2)])
def test_branch_decomposition_all_codes(a_bits, w_bits, n):
    """Sum over the M x K binary branches, weighted 2^(i+j), equals the integer dot -- for every code."""
    La, Lw = 2 ** a_bits - 1, 2 ** w_bits - 1
    ua_all = np.array(list(itertools.product(range(2 ** a_bits), repeat=n)), dtype=np.int64)
    ub_all = np.array(list(itertools.product(range(2 ** w_bits), repeat=n)), dtype=np.int64)
    acc = oracle.gemm(2 * ua_all - La, 2 * ub_all - Lw)
    step_a = max(1, len(ua_all) // 61)
    step_b = max(1, len(ub_all) // 67)
    full = len(ua_all) * len(ub_all) <= 70000
    rows = range(len(ua_all)) if full else range(0, len(ua_all), step_a)
    for r in rows:
        cols = range(len(ub_all)) if full else range(r % step_b, len(ub_all), step_b)
        for c in cols:
            assert acc[r, c] == _branch_sum(ua_all[r], ub_all[c], a_bits, w_bits)


@pytest.mark.parametrize("a_bits,w_bits", [(1, 1), (2, 2), (2, 3), (3, 3), (4, 4), (5, 2), (8, 8)])
def test_branch_decomposition_random(a_bits, w_bits):
    rng = np.random.default_rng(100 + a_bits * 8 + w_bits)
    k = 77
    ua = rng.integers(0, 2 ** a_bits, size=(9, k))
    ub = rng.integers(0, 2 ** w_bits, size=(7, k))
    acc = oracle.gemm(2 * ua - (2 ** a_bits - 1), 2 * ub - (2 ** w_bits - 1))
    for r in range(9):
        for c in range(7):
            assert acc[r, c] == _branch_sum(ua[r], ub[c], a_bits, w_bits)


@pytest.mark.parametrize("a_bits,w_bits", [(2, 2), (3, 5), (8, 8)])
def test_eq17_polynomial_equals_eq18(a_bits, w_bits):
    """Eq. 17's four-term {0,1}-encoding product, summed over a vector, equals Eq. 18 on the
    {-1,+1} integers: acc / ((2^M-1)(2^K-1))."""
    rng = np.random.default_rng(17)
    k = 40
    La, Lw = 2 ** a_bits - 1, 2 ** w_bits - 1
    ua = rng.integers(0, La + 1, size=(3, k))
    ub = rng.integers(0, Lw + 1, size=(4, k))
    acc = oracle.gemm(2 * ua - La, 2 * ub - Lw)
    out64 = oracle.scale_f64(acc, 1.0, 1.0, a_bits, w_bits)
    for r in range(3):
        for c in range(4):
            poly = Fraction(0)
            for t in range(k):
                x01, w01 = int(ua[r, t]), int(ub[c, t])
                poly += Fraction(4 * x01 * w01, La * Lw) - Fraction(2 * x01, La) - Fraction(2 * w01, Lw) + 1
            assert Fraction(int(acc[r, c]), La * Lw) == poly
            assert abs(out64[r, c] - float(poly)) <= 1e-12 * max(1.0, abs(float(poly)))


def test_one_bit_is_sign_dot():
    """At 1 x 1 bits the layer is the sign-binarised dot (Binarize = sign(HTanh(x)), sign(0) = +1)."""
    rng = np.random.default_rng(21)
    x = rng.standard_normal((12, 300)).astype(np.float32)
    w = rng.standard_normal((10, 300)).astype(np.float32)
    x[0, :5] = 0.0
    acc, _, _, _ = oracle.linear(x, w, 1, 1)
    sx = np.where(x >= 0, 1, -1).astype(np.int64)
    sw = np.where(w >= 0, 1, -1).astype(np.int64)
    assert np.array_equal(acc, sx @ sw.T)


def test_hrelu_one_bit_activations_give_weight_row_sums():
    """All activations +1 (1-bit encoder after HReLU) => acc[m][n] = sum_k q_w[n][k] for every m."""
    rng = np.random.default_rng(23)
    x = np.maximum(rng.standard_normal((5, 200)), 0).astype(np.float32)
    w = rng.standard_normal((8, 200)).astype(np.float32)
    for w_bits in (1, 2, 4):
        acc, _, _, s_w = oracle.linear(x, w, 1, w_bits)
        qw = oracle.quantize(w, s_w, w_bits).astype(np.int64)
        assert np.array_equal(acc, np.broadcast_to(qw.sum(axis=1), (5, 8)))


@pytest.mark.parametrize("bits", [1, 2, 4, 8])
def test_closed_forms(bits):
    L = 2 ** bits - 1
    k = 333
    rng = np.random.default_rng(29 + bits)
    q = 2 * rng.integers(0, L + 1, size=(4, k)) - L
    acc = oracle.gemm(q, q)
    assert np.array_equal(np.diag(acc), (q.astype(np.int64) ** 2).sum(axis=1))   # identical rows: sum q^2
    if bits == 1:
        assert np.all(np.diag(acc) == k)
    ext = np.full((2, k), L)
    ext[1] = -L
    acc = oracle.gemm(ext, ext)
    assert acc.tolist() == [[k * L * L, -k * L * L], [-k * L * L, k * L * L]]     # all-extreme codes


def test_gemm_matches_numpy_matmul():
    rng = np.random.default_rng(31)
    qa = 2 * rng.integers(0, 16, size=(33, 517)) - 15
    qb = 2 * rng.integers(0, 8, size=(29, 517)) - 7
    assert np.array_equal(oracle.gemm(qa, qb), qa.astype(np.int64) @ qb.astype(np.int64).T)


def test_gemm_int32_overflow_is_reported():
    k = 34000                                  # 255 * 255 * 34000 > 2^31
    qa = np.full((1, k), 255)
    with pytest.raises(OverflowError):
        oracle.gemm(qa, qa)


def test_scale_one_ninth():
    """Fig. 1's decoder factor at 2 x 2 bits and range 1 is 1/9 (alpha = 3, squared)."""
    acc = np.array([[9, -9, 1, 0, 27]], dtype=np.int32)
    out64 = oracle.scale_f64(acc, 1.0, 1.0, 2, 2)
    assert np.allclose(out64, [[1.0, -1.0, 1.0 / 9.0, 0.0, 3.0]], rtol=1e-15, atol=0)
    out32 = oracle.scale(acc, 1.0, 1.0, 2, 2)
    assert np.all(np.abs(out32 - out64) <= 2e-7 * np.abs(out64))


@pytest.mark.parametrize("a_bits,w_bits", [(1, 1), (2, 2), (3, 4), (8, 8)])
def test_scale_eq18_rational_and_fp32_tolerance(a_bits, w_bits):
    """Eq. 18 with ranges s_a, s_w[c]: exact rational vs the double and fp32 evaluations.
    The fp32 path (two divisions, two multiplies, one conversion) stays within 4 ulp,
    far inside the 1e-5 relative bar."""
    rng = np.random.default_rng(37)
    acc = rng.integers(-2 ** 24, 2 ** 24, size=(6, 5)).astype(np.int32)
    s_a = np.float32(3.7)
    s_w = rng.uniform(0.01, 2.0, size=5).astype(np.float32)
    La, Lw = 2 ** a_bits - 1, 2 ** w_bits - 1
    out64 = oracle.scale_f64(acc, s_a, s_w, a_bits, w_bits)
    out32 = oracle.scale(acc, s_a, s_w, a_bits, w_bits)
    for r in range(6):
        for c in range(5):
            exact = Fraction(int(acc[r, c])) * Fraction(float(s_a)) * Fraction(float(s_w[c])) / (La * Lw)
            assert abs(out64[r, c] - float(exact)) <= 1e-14 * abs(float(exact))
            assert abs(float(out32[r, c]) - float(exact)) <= 4 * 2.0 ** -24 * abs(float(exact)) * 1.01
    # per-tensor weight range = the same value for every channel
    one = oracle.scale(acc, s_a, s_w[:1], a_bits, w_bits)
    assert np.array_equal(one[:, 0], out32[:, 0])


def _im2col(q, KH, KW, stride, pad):
    """[N][C][H][W] -> [N*Ho*Wo][C*KH*KW] with explicit zeros for the border."""
    N, C, H, W = q.shape
    qp = np.zeros((N, C, H + 2 * pad, W + 2 * pad), dtype=np.int64)
    qp[:, :, pad:pad + H, pad:pad + W] = q
    Ho = (H + 2 * pad - KH) // stride + 1
    Wo = (W + 2 * pad - KW) // stride + 1
    cols = np.empty((N, Ho, Wo, C, KH, KW), dtype=np.int64)
    for oh in range(Ho):
        for ow in range(Wo):
            cols[:, oh, ow] = qp[:, :, oh * stride:oh * stride + KH, ow * stride:ow * stride + KW]
    return cols.reshape(N * Ho * Wo, C * KH * KW), Ho, Wo


@pytest.mark.parametrize("KH,stride,pad", [(1, 1, 0), (1, 2, 0), (3, 1, 0), (3, 1, 1), (3, 2, 1)])
def test_conv_equals_matmul_on_materialised_im2col(KH, stride, pad):
    rng = np.random.default_rng(41 + KH + stride + pad)
    N, C, H, W, O = 2, 5, 9, 8, 6
    qx = 2 * rng.integers(0, 8, size=(N, C, H, W)) - 7
    qw = 2 * rng.integers(0, 4, size=(O, C, KH, KH)) - 3
    acc = oracle.conv(qx, qw, stride, pad)
    cols, Ho, Wo = _im2col(qx, KH, KH, stride, pad)
    ref = (cols @ qw.reshape(O, -1).astype(np.int64).T).reshape(N, Ho, Wo, O).transpose(0, 3, 1, 2)
    assert acc.shape == (N, O, Ho, Wo)
    assert np.array_equal(acc, ref)
    # single-element sampler agrees with the full loop
    for (b, o, oh, ow) in [(0, 0, 0, 0), (1, O - 1, Ho - 1, Wo - 1), (1, 2, Ho // 2, 0)]:
        assert oracle.conv_at(qx, qw, stride, pad, b, o, oh, ow) == ref[b, o, oh, ow]


def test_conv_sliding_window_einsum():
    """Against numpy's sliding_window_view + einsum (a library routine the oracle does not use)."""
    rng = np.random.default_rng(43)
    qx = 2 * rng.integers(0, 4, size=(3, 4, 7, 7)) - 3
    qw = 2 * rng.integers(0, 4, size=(5, 4, 3, 3)) - 3
    win = np.lib.stride_tricks.sliding_window_view(qx.astype(np.int64), (3, 3), axis=(2, 3))
    ref = np.einsum("nchwij,ocij->nohw", win, qw.astype(np.int64))
    assert np.array_equal(oracle.conv(qx, qw, 1, 0), ref)


def test_conv_zero_padding_contributes_nothing():
    """pad=1 equals pad=0 on a border of explicit zeros, and a corner output sums only its 4 valid taps."""
    rng = np.random.default_rng(47)
    qx = 2 * rng.integers(0, 2, size=(1, 3, 5, 5)) - 1
    qw = np.ones((2, 3, 3, 3), dtype=np.int64)
    acc = oracle.conv(qx, qw, 1, 1)
    assert acc[0, 0, 0, 0] == qx[0, :, 0:2, 0:2].sum()
    qp = np.zeros((1, 3, 7, 7), dtype=np.int64)
    qp[:, :, 1:6, 1:6] = qx
    assert np.array_equal(acc, oracle.conv(qp, qw, 1, 0))


def test_stride_two_is_subsampled_stride_one():
    rng = np.random.default_rng(53)
    qx = 2 * rng.integers(0, 4, size=(2, 3, 9, 9)) - 3
    qw = 2 * rng.integers(0, 4, size=(4, 3, 3, 3)) - 3
    assert np.array_equal(oracle.conv(qx, qw, 2, 1), oracle.conv(qx, qw, 1, 1)[:, :, ::2, ::2])


def test_layer_helpers_compose_the_steps():
    rng = np.random.default_rng(59)
    x = np.maximum(rng.standard_normal((4, 64)), 0).astype(np.float32)
    w = (rng.standard_normal((6, 64)) * 0.01).astype(np.float32)
    acc, out, s_a, s_w = oracle.linear(x, w, 2, 2, w_per_row=True)
    assert s_a[0] == np.abs(x).max() and np.array_equal(s_w, np.abs(w).max(axis=1))
    qa = oracle.quantize(x, s_a, 2).astype(np.int64)
    qb = oracle.quantize(w, s_w, 2, per_row=True).astype(np.int64)
    assert np.array_equal(acc, qa @ qb.T)
    ref = acc.astype(np.float64) * float(s_a[0]) * s_w.astype(np.float64)[None, :] / 9.0
    assert np.all(np.abs(out - ref) <= 1e-6 * np.abs(ref))


@pytest.mark.parametrize("a_bits,w_bits", [(2, 2), (4, 3)])
def test_scale_on_nchw_accumulators(a_bits, w_bits):
    """The decoder scale on a convolution's [N][O][Ho][Wo] accumulators: the weight range of
    output channel o multiplies every pixel of channel o and nothing else.  Checked element by
    element against Eq. 18 in exact rationals, and against the 2-D path applied per channel."""
    rng = np.random.default_rng(67)
    N, O, Ho, Wo = 3, 5, 4, 6
    acc = rng.integers(-2 ** 20, 2 ** 20, size=(N, O, Ho, Wo)).astype(np.int32)
    s_a = np.float32(1.9)
    s_w = rng.uniform(0.05, 3.0, size=O).astype(np.float32)     # all different: a wrong channel index shows
    La, Lw = 2 ** a_bits - 1, 2 ** w_bits - 1
    out32 = oracle.scale(acc, s_a, s_w, a_bits, w_bits)
    out64 = oracle.scale_f64(acc, s_a, s_w, a_bits, w_bits)
    assert out32.shape == acc.shape and out64.shape == acc.shape
    for idx in np.ndindex(N, O, Ho, Wo):
        exact = Fraction(int(acc[idx])) * Fraction(float(s_a)) * Fraction(float(s_w[idx[1]])) / (La * Lw)
        assert abs(out64[idx] - float(exact)) <= 1e-14 * abs(float(exact))
        assert abs(float(out32[idx]) - float(exact)) <= 4 * 2.0 ** -24 * abs(float(exact)) * 1.01
    # the 2-D path (rows = pixels, columns = channels) gives the same bits
    flat = acc.transpose(0, 2, 3, 1).reshape(-1, O)
    ref2d = oracle.scale(flat, s_a, s_w, a_bits, w_bits).reshape(N, Ho, Wo, O).transpose(0, 3, 1, 2)
    assert np.array_equal(out32, ref2d)
    # one weight range for the whole tensor
    one = oracle.scale(acc, s_a, s_w[2:3], a_bits, w_bits)
    assert np.array_equal(one[:, 2], out32[:, 2])


@pytest.mark.parametrize("per_channel", [True, False])
@pytest.mark.parametrize("act", [oracle.HTANH, oracle.HRELU])
def test_conv_layer_composes_the_steps(per_channel, act):
    """The whole encoded convolution layer against its parts put together by hand: numpy ranges,
    the (separately pinned) quantizer, a matmul on a materialised im2col, Eq. 18 in rationals."""
    rng = np.random.default_rng(71 + int(per_channel) + 2 * act)
    N, C, H, W, O, a_bits, w_bits, stride, pad = 2, 6, 7, 5, 4, 3, 2, 2, 1
    x = rng.standard_normal((N, C, H, W)).astype(np.float32)
    w = (rng.standard_normal((O, C, 3, 3)) * rng.uniform(0.1, 2.0, size=(O, 1, 1, 1))).astype(np.float32)
    acc, out, s_a, s_w = oracle.conv_layer(x, w, a_bits, w_bits, stride, pad, per_channel, act)
    ref_sa = np.nanmax(np.maximum(x, 0)) if act == oracle.HRELU else np.nanmax(np.abs(x))
    ref_sw = np.abs(w).reshape(O, -1).max(axis=1) if per_channel else np.abs(w).max(keepdims=True).reshape(1)
    assert s_a.shape == (1,) and s_a[0] == ref_sa
    assert np.array_equal(s_w, ref_sw)
    qx = oracle.quantize(x, ref_sa, a_bits, act=act).astype(np.int64)
    qw = np.stack([oracle.quantize(w[o], ref_sw[o if per_channel else 0], w_bits) for o in range(O)]).astype(np.int64)
    if act == oracle.HRELU:
        assert qx.min() >= 1                                     # the negative side sits on the level above zero
    cols, Ho, Wo = _im2col(qx, 3, 3, stride, pad)
    ref = (cols @ qw.reshape(O, -1).T).reshape(N, Ho, Wo, O).transpose(0, 3, 1, 2)
    assert np.array_equal(acc, ref)
    La, Lw = 2 ** a_bits - 1, 2 ** w_bits - 1
    for idx in np.ndindex(*acc.shape):
        sw = ref_sw[idx[1] if per_channel else 0]
        exact = Fraction(int(ref[idx])) * Fraction(float(ref_sa)) * Fraction(float(sw)) / (La * Lw)
        assert abs(float(out[idx]) - float(exact)) <= 4 * 2.0 ** -24 * abs(float(exact)) * 1.01


def test_epilogue_is_one_rounded_add_each():
    """Bias, residual and max(., 0) after the decoder: each add rounds once in fp32, in that order."""
    out = np.array([[1.0, -2.0, 3.0], [0.5, 16777216.0, -1.0]], dtype=np.float32)
    bias = np.array([0.25, 1.0, -4.0], dtype=np.float32)
    res = np.array([[1.0, 1.0, 1.0], [-1.0, 1.0, 0.5]], dtype=np.float32)
    got = oracle.epilogue(out, bias, res, relu=True)
    # 16777216 + 1 rounds back to 16777216 (tie to even), then + 1 does so again: two roundings, not one exact sum
    assert got.tolist() == [[2.25, 0.0, 0.0], [0.0, 16777216.0, 0.0]]
    assert oracle.epilogue(out, None, None, False).tolist() == out.tolist()
    assert oracle.epilogue(out, bias).tolist() == [[1.25, -1.0, -1.0], [0.75, 16777216.0, -5.0]]
    nchw = np.zeros((1, 3, 2, 2), dtype=np.float32)
    assert oracle.epilogue(nchw, bias)[0, :, 1, 1].tolist() == bias.tolist()
    rng = np.random.default_rng(89)
    a, b, r = (rng.standard_normal((5, 7)).astype(np.float32) for _ in range(3))
    ref = np.maximum(np.float32(1) * ((a.astype(np.float64) + b[0].astype(np.float64)).astype(np.float32).astype(np.float64)
                                      + r.astype(np.float64)).astype(np.float32), 0)
    assert np.array_equal(oracle.epilogue(a, b[0], r, True), ref)
