"""GPU parity of the deconvolution (transposed convolution) on packed planes against the CPU oracle.

The oracle spreads every input pixel over its output window; the library gathers, per output phase,
through the branch kernel.  int32 accumulators bit-exact, fp32 outputs within 1e-5 relative; the
packed filter phases are unpacked on the test side and compared with the oracle's codes."""
import numpy as np
import pytest
import torch

import oracle
from paper_1905_13389_b200 import inputs
from tests._util import rel_close, unpack_planes

pytestmark = pytest.mark.gpu

FILTERS = [(4, 4, 2, 1), (2, 2, 2, 0), (3, 3, 2, 1), (3, 3, 2, 0), (4, 4, 2, 0), (3, 3, 1, 1), (4, 4, 1, 2),
           (2, 3, 2, 1), (4, 2, 2, 0), (1, 1, 1, 0), (2, 2, 1, 1), (4, 3, 2, 2)]


def _dev(a, cuda):
    return torch.from_numpy(np.ascontiguousarray(a)).to(cuda)


def _run(mpq, cuda, x, w, a_bits, w_bits, stride, pad, per_channel, act, **glue):
    N, C, H, W = x.shape
    O, _, KH, KW = w.shape
    xd, wd = _dev(x, cuda), _dev(w, cuda)
    mode = mpq.SCALE_PER_ROW if per_channel else mpq.SCALE_PER_TENSOR
    sa, sw = mpq.absmax(xd, 0, act), mpq.absmax(wd, mode)
    xp = mpq.encode_nchw(xd, sa, a_bits, act)
    wp, taps = mpq.encode_deconv_weights(wd, sw, w_bits, stride, mode)
    Ho, Wo = (H - 1) * stride - 2 * pad + KH, (W - 1) * stride - 2 * pad + KW
    yi = torch.full((N, O, Ho, Wo), -7, dtype=torch.int32, device=cuda)
    yf = torch.full((N, O, Ho, Wo), float("nan"), dtype=torch.float32, device=cuda)
    mpq.deconv(xp, a_bits, N, C, H, W, wp, w_bits, taps, O, KH, KW, stride, pad, yi, yf, sa, sw, mode, **glue)
    torch.cuda.synchronize()
    return yi.cpu().numpy(), yf.cpu().numpy(), wp, taps


@pytest.mark.parametrize("KH,KW,stride,pad", FILTERS)
def test_deconv_every_filter_shape(mpq, cuda, KH, KW, stride, pad):
    a_bits, w_bits = 2, 3
    N, C, H, W, O = 3, 64, 9, 7, 40                      # 189 input pixels: several tiles per phase, ragged
    x = inputs.uniform_levels(30, KH * 10 + KW, (N, C, H, W), a_bits)
    w = inputs.uniform_levels(30, 100 + stride * 10 + pad, (O, C, KH, KW), w_bits)
    acc_ref, out_ref, _, _ = oracle.deconv_layer(x, w, a_bits, w_bits, stride, pad, True, oracle.HRELU)
    yi, yf, _, _ = _run(mpq, cuda, x, w, a_bits, w_bits, stride, pad, True, mpq.ACT_HRELU)
    assert np.array_equal(yi, acc_ref)
    assert rel_close(yf, out_ref)
    assert np.unique(acc_ref).size > 8


@pytest.mark.parametrize("stride,KH", [(2, 4), (2, 3), (1, 3)])
def test_deconv_weight_phases_and_tap_sums(mpq, cuda, stride, KH):
    """The packed filter: per phase (kh mod stride, kw mod stride) a matrix whose row o lists that phase's
    taps (t_h, t_w, c); tap sums counted in the same order."""
    bits, O, C, KW = 3, 5, 64, KH
    w = inputs.uniform_levels(31, stride * 10 + KH, (O, C, KH, KW), bits)
    s_w = oracle.absmax(w, True)
    qw = oracle.quantize(w, s_w, bits, per_row=True)
    u = oracle.levels(qw, bits)
    wd = _dev(w, cuda)
    planes, taps = mpq.encode_deconv_weights(wd, mpq.absmax(wd, mpq.SCALE_PER_ROW), bits, stride)
    planes, taps = planes.cpu().numpy(), taps.cpu().numpy()
    at, tap = 0, 0
    for r_h in range(stride):
        for r_w in range(stride):
            khs, kws = list(range(r_h, KH, stride)), list(range(r_w, KW, stride))
            K = len(khs) * len(kws) * C
            rw = mpq.row_words(K)
            got = unpack_planes(planes[at:at + bits * O * rw].reshape(bits, O, rw), K)
            want = np.stack([u[:, :, kh, kw] for kh in khs for kw in kws], axis=1).reshape(O, K)
            assert np.array_equal(got, want), (r_h, r_w)
            for kh in khs:
                for kw in kws:
                    assert np.array_equal(taps[tap], qw[:, :, kh, kw].astype(np.int64).sum(axis=1)), (kh, kw)
                    tap += 1
            at += bits * O * rw
    assert at == planes.size and tap == KH * KW


@pytest.mark.parametrize("seed", range(20))
def test_deconv_random_cases(mpq, cuda, seed):
    rng = np.random.default_rng(5000 + seed)
    a_bits, w_bits = int(rng.integers(1, 9)), int(rng.integers(1, 9))
    C = int(rng.choice([32, 64, 128, 256]))
    stride = int(rng.choice([1, 2, 2]))
    KH, KW = int(rng.integers(stride, 5)), int(rng.integers(stride, 5))
    pad = int(rng.integers(0, min(KH, KW)))
    H, W = int(rng.integers(1, 14)), int(rng.integers(1, 14))
    if (H - 1) * stride - 2 * pad + KH <= 0 or (W - 1) * stride - 2 * pad + KW <= 0:
        pad = 0
    N = int(rng.choice([1, 2, 5]))
    O = int(rng.choice([1, 7, 32, 33, 80]))
    if a_bits + w_bits > 12 and C > 128:                 # keep taps * C * L_a * L_w inside int32
        C = 128
    act, per_channel = int(rng.integers(0, 2)), bool(rng.integers(0, 2))
    x = inputs.uniform_levels(32, 2 * seed, (N, C, H, W), a_bits)
    w = inputs.uniform_levels(32, 2 * seed + 1, (O, C, KH, KW), w_bits) * np.float32(1 + seed)
    acc_ref, out_ref, _, _ = oracle.deconv_layer(x, w, a_bits, w_bits, stride, pad, per_channel, act)
    yi, yf, _, _ = _run(mpq, cuda, x, w, a_bits, w_bits, stride, pad, per_channel, act)
    case = (a_bits, w_bits, C, KH, KW, stride, pad, H, W, N, O)
    assert np.array_equal(yi, acc_ref), case
    assert rel_close(yf, out_ref), case


def test_deconv_glue_in_the_store(mpq, cuda):
    """Residual add, max(., 0) and the next encoder's range ride in the store, as for the convolution."""
    a_bits, w_bits, stride, pad = 4, 4, 2, 1
    N, C, H, W, O, KH = 2, 128, 6, 5, 64, 4
    x = inputs.normal(33, 0, (N, C, H, W), relu=True)
    w = inputs.normal(33, 1, (O, C, KH, KH))
    acc_ref, out_ref, _, _ = oracle.deconv_layer(x, w, a_bits, w_bits, stride, pad, True, oracle.HRELU)
    res = inputs.normal(33, 2, out_ref.shape)
    want = oracle.epilogue(out_ref, None, res, True)
    out_max = torch.zeros(1, dtype=torch.float32, device=cuda)
    yi, yf, _, _ = _run(mpq, cuda, x, w, a_bits, w_bits, stride, pad, True, mpq.ACT_HRELU,
                        residual=_dev(res, cuda), relu=True, out_max=out_max)
    assert np.array_equal(yi, acc_ref)
    assert rel_close(yf, want)
    assert float(out_max.item()) == float(yf.max())


def test_deconv_upsampling_layer_sampled(mpq, cuda):
    """A generator-sized layer (W4A4, 4 x 4 stride 2 pad 1, 256 -> 128 channels, 28 -> 56 pixels, batch 32),
    the launch configuration that is timed: the oracle's gather over sampled outputs, borders included."""
    a_bits, w_bits, stride, pad = 4, 4, 2, 1
    N, C, H, W, O, KH = 32, 256, 28, 28, 128, 4
    x = inputs.normal(34, 0, (N, C, H, W), relu=True)
    w = inputs.normal(34, 1, (O, C, KH, KH), std=0.05)
    yi, yf, _, _ = _run(mpq, cuda, x, w, a_bits, w_bits, stride, pad, True, mpq.ACT_HRELU)
    s_a, s_w = oracle.absmax(x, False, oracle.HRELU), oracle.absmax(w, True)
    qx = oracle.quantize(x, s_a, a_bits, act=oracle.HRELU)
    qw = oracle.quantize(w, s_w, w_bits, per_row=True)
    Ho = (H - 1) * stride - 2 * pad + KH
    assert yi.shape == (N, O, Ho, Ho) and Ho == 56
    rng = np.random.default_rng(9)
    pts = [(0, 0, 0, 0), (N - 1, O - 1, Ho - 1, Ho - 1), (1, 2, 0, Ho - 1), (2, 3, Ho - 1, 0), (3, 5, 1, 1), (4, 7, 54, 55)]
    pts += [tuple(int(v) for v in (rng.integers(N), rng.integers(O), rng.integers(Ho), rng.integers(Ho))) for _ in range(60)]
    for (b, o, oh, ow) in pts:
        # one image, one output channel: the oracle's deconvolution on that slice
        acc = oracle.deconv(qx[b:b + 1], qw[o:o + 1], stride, pad)[0, 0, oh, ow]
        assert int(yi[b, o, oh, ow]) == int(acc), (b, o, oh, ow)
        ref = oracle.scale(np.array([[acc]], np.int32), s_a[0], s_w[o:o + 1], a_bits, w_bits)[0, 0]
        assert abs(float(yf[b, o, oh, ow]) - float(ref)) <= 1e-5 * abs(float(ref))


def test_deconv_rejects_what_it_does_not_support(mpq, cuda):
    xp = torch.zeros((2, 1, 4, 4, 1), dtype=torch.int32, device=cuda)
    wp = torch.zeros((4096,), dtype=torch.int32, device=cuda)
    taps = torch.zeros((25, 8), dtype=torch.int32, device=cuda)
    yi = torch.zeros((1, 8, 16, 16), dtype=torch.int32, device=cuda)
    from paper_1905_13389_b200.binding import MpqError
    for (KH, KW, stride, pad) in [(5, 5, 2, 1), (1, 1, 2, 0), (3, 3, 3, 0), (3, 3, 2, 3), (2, 2, 2, -1)]:
        with pytest.raises(MpqError):
            mpq.deconv(xp, 2, 1, 32, 4, 4, wp, 2, taps, 8, KH, KW, stride, pad, yi, None)
    with pytest.raises(MpqError):
        mpq.deconv(xp, 2, 1, 32, 4, 4, wp, 2, taps, 8, 4, 4, 2, 1, None, None)       # no output buffer
    with pytest.raises(MpqError):
        mpq.encode_deconv_weights(torch.zeros((8, 32, 5, 5), device=cuda), torch.ones(8, device=cuda), 2, 2)
    assert not yi.any()
