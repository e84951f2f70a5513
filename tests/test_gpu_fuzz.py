"""Seeded random sweeps of the product kernels against the CPU oracle: shapes, bit-widths, strides
and paddings drawn at random (every tile width, ragged tiles, short and half-filled k, single rows),
all levels present in the operands.  int32 bit-exact, fp32 within 1e-5 relative."""
import numpy as np
import pytest
import torch

import oracle
from paper_1905_13389_b200 import inputs
from tests._util import rel_close

pytestmark = pytest.mark.gpu


def _dev(a, cuda):
    return torch.from_numpy(np.ascontiguousarray(a)).to(cuda)


@pytest.mark.parametrize("seed", range(24))
def test_gemm_random_cases(mpq, cuda, seed):
    rng = np.random.default_rng(1000 + seed)
    a_bits, w_bits = int(rng.integers(1, 9)), int(rng.integers(1, 9))
    m = int(rng.choice([1, 3, 17, 64, 65, 200, 513]))
    n = int(rng.choice([1, 2, 31, 100, 128, 129, 700, 2500]))
    k = int(rng.choice([1, 31, 32, 33, 127, 128, 129, 500, 1024, 3000]))
    per_row = bool(rng.integers(0, 2))
    act = int(rng.integers(0, 2))
    x = inputs.uniform_levels(20, 2 * seed, (m, k), a_bits)
    w = inputs.uniform_levels(20, 2 * seed + 1, (n, k), w_bits) * np.float32(0.5 + seed)
    acc_ref, out_ref, s_a, s_w = oracle.linear(x, w, a_bits, w_bits, w_per_row=per_row, a_act=act)
    xd, wd = _dev(x, cuda), _dev(w, cuda)
    sa_d, sw_d = mpq.absmax(xd, 0, act), mpq.absmax(wd, int(per_row))
    ap, wp = mpq.encode(xd, sa_d, a_bits, 0, act), mpq.encode(wd, sw_d, w_bits, int(per_row))
    ci = torch.full((m, n), -5, dtype=torch.int32, device=cuda)
    cf = torch.full((m, n), float("nan"), dtype=torch.float32, device=cuda)
    mpq.gemm(ap, a_bits, wp, w_bits, m, n, k, ci, cf, sa_d, sw_d, int(per_row))
    assert np.array_equal(ci.cpu().numpy(), acc_ref), (a_bits, w_bits, m, n, k)
    assert rel_close(cf.cpu().numpy(), out_ref), (a_bits, w_bits, m, n, k)


@pytest.mark.parametrize("seed", range(24))
def test_conv_random_cases(mpq, cuda, seed):
    rng = np.random.default_rng(2000 + seed)
    a_bits, w_bits = int(rng.integers(1, 9)), int(rng.integers(1, 9))
    C = int(rng.choice([32, 64, 128, 256, 384]))
    ksz = int(rng.choice([1, 3]))
    stride = int(rng.choice([1, 2]))
    pad = int(rng.integers(0, 2)) if ksz == 3 else 0
    H = int(rng.integers(3, 20))
    W = int(rng.integers(3, 20))
    N = int(rng.choice([1, 2, 5, 9]))
    O = int(rng.choice([1, 7, 32, 33, 80]))
    if a_bits + w_bits > 12 and C > 128:          # keep 9 * C * L_a * L_w inside int32
        C = 128
    act = int(rng.integers(0, 2))
    x = inputs.uniform_levels(21, 2 * seed, (N, C, H, W), a_bits)
    w = inputs.uniform_levels(21, 2 * seed + 1, (O, C, ksz, ksz), w_bits)
    acc_ref, out_ref, s_a, s_w = oracle.conv_layer(x, w, a_bits, w_bits, stride, pad, True, act)
    xd, wd = _dev(x, cuda), _dev(w, cuda)
    sa_d, sw_d = mpq.absmax(xd, 0, act), mpq.absmax(wd, mpq.SCALE_PER_ROW)
    xp = mpq.encode_nchw(xd, sa_d, a_bits, act)
    wp, taps = mpq.encode_oihw(wd, sw_d, w_bits, mpq.SCALE_PER_ROW)
    yi = torch.full(acc_ref.shape, -5, dtype=torch.int32, device=cuda)
    yf = torch.full(acc_ref.shape, float("nan"), dtype=torch.float32, device=cuda)
    mpq.conv(xp, a_bits, N, C, H, W, wp, w_bits, taps, O, ksz, ksz, stride, pad, yi, yf, sa_d, sw_d, mpq.SCALE_PER_ROW)
    key = (a_bits, w_bits, N, C, H, W, O, ksz, stride, pad)
    assert np.array_equal(yi.cpu().numpy(), acc_ref), key
    assert rel_close(yf.cpu().numpy(), out_ref), key


def test_gemm_very_tall_and_very_wide(mpq, cuda):
    """Grid extremes: 200 000 rows against a handful of columns, and the transpose of that shape."""
    for (m, n) in ((200000, 5), (5, 200000)):
        k = 96
        x = inputs.uniform_levels(22, m % 7, (m, k), 2)
        w = inputs.uniform_levels(22, 10 + n % 7, (n, k), 3)
        acc_ref, out_ref, s_a, s_w = oracle.linear(x, w, 2, 3, w_per_row=False)
        xd, wd = _dev(x, cuda), _dev(w, cuda)
        sa_d, sw_d = mpq.absmax(xd), mpq.absmax(wd)
        ci = torch.empty((m, n), dtype=torch.int32, device=cuda)
        cf = torch.empty((m, n), dtype=torch.float32, device=cuda)
        mpq.gemm(mpq.encode(xd, sa_d, 2), 2, mpq.encode(wd, sw_d, 3), 3, m, n, k, ci, cf, sa_d, sw_d)
        assert np.array_equal(ci.cpu().numpy(), acc_ref)
        assert rel_close(cf.cpu().numpy(), out_ref)


def test_two_streams_run_independent_layers(mpq, cuda):
    """The entry points keep no hidden state between calls: two different layers issued alternately on
    two side streams (so that their kernels interleave on the device) give the oracle's results."""
    cases = []
    for t, (m, n, k, ab, wb) in enumerate(((300, 500, 2000, 2, 2), (257, 390, 1500, 4, 3))):
        x = inputs.uniform_levels(23, 2 * t, (m, k), ab)
        w = inputs.uniform_levels(23, 2 * t + 1, (n, k), wb)
        acc_ref, out_ref, _, _ = oracle.linear(x, w, ab, wb, w_per_row=True)
        cases.append(dict(x=_dev(x, cuda), w=_dev(w, cuda), ab=ab, wb=wb, acc=acc_ref, out=out_ref,
                          oi=torch.empty((m, n), dtype=torch.int32, device=cuda),
                          of=torch.empty((m, n), dtype=torch.float32, device=cuda),
                          stream=torch.cuda.Stream()))
    torch.cuda.synchronize()
    for _ in range(6):
        for c in cases:
            with torch.cuda.stream(c["stream"]):
                mpq.linear(c["x"], c["w"], c["ab"], c["wb"], mpq.ACT_HTANH, mpq.SCALE_PER_ROW, c["oi"], c["of"])
    torch.cuda.synchronize()
    for c in cases:
        assert np.array_equal(c["oi"].cpu().numpy(), c["acc"])
        assert rel_close(c["of"].cpu().numpy(), c["out"])


def _pack_nhwc(u, bits):
    """Level indices [N][O][Ho][Wo] -> planes [bits][N][Ho][Wo][O/32] (test-side packer)."""
    N, O, Ho, Wo = u.shape
    t = u.transpose(0, 2, 3, 1).reshape(N, Ho, Wo, O // 32, 32).astype(np.uint64)
    weights = np.uint64(1) << np.arange(32, dtype=np.uint64)
    return np.stack([(((t >> np.uint64(p)) & np.uint64(1)) * weights).sum(axis=4).astype(np.uint32) for p in range(bits)])


@pytest.mark.parametrize("seed", range(16))
def test_gemm_fused_random_cases(mpq, cuda, seed):
    """The glue in the GEMM store (bias, residual, max in any combination) on random shapes, among them
    few-tile / long-k shapes that run with k-groups inside the CTA."""
    rng = np.random.default_rng(3000 + seed)
    a_bits, w_bits = int(rng.integers(1, 9)), int(rng.integers(1, 9))
    m = int(rng.choice([1, 17, 64, 100]))
    n = int(rng.choice([3, 100, 1000, 2500, 4096]))
    k = int(rng.choice([129, 1024, 3000, 9216, 20000]))
    while (2 ** a_bits - 1) * (2 ** w_bits - 1) * k >= 2 ** 31:
        k //= 2
    per_row = bool(rng.integers(0, 2))
    x = inputs.uniform_levels(24, 2 * seed, (m, k), a_bits)
    w = inputs.uniform_levels(24, 2 * seed + 1, (n, k), w_bits)
    acc_ref, out_ref, _, _ = oracle.linear(x, w, a_bits, w_bits, w_per_row=per_row)
    scale = float(np.abs(out_ref).max()) or 1.0
    bias = (rng.standard_normal(n) * 0.3 * scale).astype(np.float32) if rng.integers(0, 2) else None
    res = (rng.standard_normal((m, n)) * 0.3 * scale).astype(np.float32) if rng.integers(0, 2) else None
    relu = bool(rng.integers(0, 2))
    ref = oracle.epilogue(out_ref, bias, res, relu)
    xd, wd = _dev(x, cuda), _dev(w, cuda)
    sa_d, sw_d = mpq.absmax(xd), mpq.absmax(wd, int(per_row))
    ap, wp = mpq.encode(xd, sa_d, a_bits), mpq.encode(wd, sw_d, w_bits, int(per_row))
    ci = torch.full((m, n), -5, dtype=torch.int32, device=cuda)
    cf = torch.full((m, n), float("nan"), dtype=torch.float32, device=cuda)
    mpq.gemm_fused(ap, a_bits, wp, w_bits, m, n, k, ci, cf, sa_d, sw_d, int(per_row),
                   None if bias is None else _dev(bias, cuda), None if res is None else _dev(res, cuda), relu)
    key = (a_bits, w_bits, m, n, k, per_row, bias is not None, res is not None, relu)
    assert np.array_equal(ci.cpu().numpy(), acc_ref), key
    assert rel_close(cf.cpu().numpy(), ref), key


@pytest.mark.parametrize("seed", range(16))
def test_conv_encoded_random_cases(mpq, cuda, seed):
    """The consumer's Encoder in the convolution's store on random layers: planes equal the oracle's codes
    of the oracle's (glued) fp32 output under a range fixed beforehand."""
    rng = np.random.default_rng(4000 + seed)
    a_bits, w_bits, next_bits = int(rng.integers(1, 9)), int(rng.integers(1, 9)), int(rng.integers(1, 9))
    C = int(rng.choice([32, 64, 128, 256]))
    ksz = int(rng.choice([1, 3]))
    stride = int(rng.choice([1, 2]))
    pad = int(rng.integers(0, 2)) if ksz == 3 else 0
    H, W = int(rng.integers(3, 16)), int(rng.integers(3, 16))
    N = int(rng.choice([1, 2, 5]))
    O = int(rng.choice([32, 64, 96, 160]))
    if a_bits + w_bits > 12 and C > 128:
        C = 128
    x = inputs.uniform_levels(25, 2 * seed, (N, C, H, W), a_bits)
    w = inputs.uniform_levels(25, 2 * seed + 1, (O, C, ksz, ksz), w_bits)
    acc_ref, out_ref, _, _ = oracle.conv_layer(x, w, a_bits, w_bits, stride, pad, True, oracle.HTANH)
    res = (rng.standard_normal(out_ref.shape) * 0.4 * np.abs(out_ref).max()).astype(np.float32) if rng.integers(0, 2) else None
    relu = bool(rng.integers(0, 2))
    act = int(rng.integers(0, 2))
    ref = oracle.epilogue(out_ref, None, res, relu)
    s_next = np.array([rng.uniform(0.3, 1.2) * max(float(np.abs(ref).max()), 1e-6)], np.float32)
    want = _pack_nhwc(oracle.levels(oracle.quantize(ref, s_next, next_bits, act=act), next_bits), next_bits)
    xd, wd = _dev(x, cuda), _dev(w, cuda)
    sa_d, sw_d = mpq.absmax(xd), mpq.absmax(wd, mpq.SCALE_PER_ROW)
    xp = mpq.encode_nchw(xd, sa_d, a_bits)
    wp, taps = mpq.encode_oihw(wd, sw_d, w_bits, mpq.SCALE_PER_ROW)
    keep = bool(rng.integers(0, 2))
    yf = torch.full(acc_ref.shape, float("nan"), dtype=torch.float32, device=cuda) if keep else None
    planes = mpq.conv_encoded(xp, a_bits, N, C, H, W, wp, w_bits, taps, O, ksz, ksz, stride, pad, None, yf, sa_d, sw_d,
                              mpq.SCALE_PER_ROW, None if res is None else _dev(res, cuda), relu, None,
                              _dev(s_next, cuda), act, next_bits)
    key = (a_bits, w_bits, next_bits, N, C, H, W, O, ksz, stride, pad, res is not None, relu, act)
    assert np.array_equal(planes.cpu().numpy().view(np.uint32), want), key
    if keep:
        assert np.array_equal(yf.cpu().numpy(), ref), key


@pytest.mark.parametrize("a_bits,w_bits,m,n,k", [
    (2, 2, 64, 4090, 6144),      # 128 tiles of 32 columns, the last one 26 wide
    (1, 1, 64, 4096, 12288),     # two k-quads per group
    (4, 4, 64, 2044, 3200),      # two held tiles x 64
    (8, 3, 33, 1000, 4096),      # 16-row held tiles, two k-groups
    (2, 2, 64, 28, 6144),        # a single tile
])
def test_gemm_small_batch_k_group_shapes(mpq, cuda, a_bits, w_bits, m, n, k):
    """Small-batch layers with at most one tile per multiprocessor (two or three k-groups per CTA):
    ragged last tiles, every held-tile height, both outputs, glue in the store."""
    x = inputs.uniform_levels(22, m + n, (m, k), a_bits)
    w = inputs.uniform_levels(22, k, (n, k), w_bits)
    acc_ref, out_ref, s_a, s_w = oracle.linear(x, w, a_bits, w_bits, w_per_row=True, a_act=oracle.HRELU)
    bias = inputs.normal(22, 7, (n,))
    want = oracle.epilogue(out_ref, bias, None, True)
    xd, wd = _dev(x, cuda), _dev(w, cuda)
    sa_d, sw_d = mpq.absmax(xd, 0, mpq.ACT_HRELU), mpq.absmax(wd, mpq.SCALE_PER_ROW)
    ap, wp = mpq.encode(xd, sa_d, a_bits, 0, mpq.ACT_HRELU), mpq.encode(wd, sw_d, w_bits, mpq.SCALE_PER_ROW)
    ci = torch.full((m, n), -5, dtype=torch.int32, device=cuda)
    cf = torch.full((m, n), float("nan"), dtype=torch.float32, device=cuda)
    mpq.gemm(ap, a_bits, wp, w_bits, m, n, k, ci, cf, sa_d, sw_d, mpq.SCALE_PER_ROW)
    assert np.array_equal(ci.cpu().numpy(), acc_ref)
    assert rel_close(cf.cpu().numpy(), out_ref)
    cf.fill_(float("nan"))
    mpq.gemm_fused(ap, a_bits, wp, w_bits, m, n, k, None, cf, sa_d, sw_d, mpq.SCALE_PER_ROW, _dev(bias, cuda), None, True)
    assert rel_close(cf.cpu().numpy(), want)


@pytest.mark.parametrize("C", [32, 64, 128, 256])
@pytest.mark.parametrize("a_bits,w_bits,stride", [(4, 4, 2), (1, 1, 1), (8, 8, 2), (3, 5, 1), (2, 7, 2)])
def test_pointwise_conv_small_channel_counts(mpq, cuda, C, a_bits, w_bits, stride):
    """1 x 1 convolutions over at most 256 channels (the shortcut convolutions of a residual stack): one
    thread per output pixel, output channels in blocks of 32.  Ragged pixel and channel counts, both
    outputs, residual + max(., 0) + the next encoder's range in the store; per-tensor weight range too."""
    N, H, W, O = 3, 13, 11, 72                        # 3 * 7 * 6 = 126 or 429 pixels, 72 = 2 * 32 + 8 channels
    if a_bits + w_bits > 12:
        O = 40
    x = inputs.uniform_levels(24, C + stride, (N, C, H, W), a_bits)
    w = inputs.uniform_levels(24, 100 + C, (O, C, 1, 1), w_bits) * np.float32(0.37)
    for per_channel in (True, False):
        acc_ref, out_ref, s_a, s_w = oracle.conv_layer(x, w, a_bits, w_bits, stride, 0, per_channel, oracle.HRELU)
        res = inputs.normal(24, 7, out_ref.shape)
        want = oracle.epilogue(out_ref, None, res, True)
        xd, wd = _dev(x, cuda), _dev(w, cuda)
        mode = mpq.SCALE_PER_ROW if per_channel else mpq.SCALE_PER_TENSOR
        sa_d, sw_d = mpq.absmax(xd, 0, mpq.ACT_HRELU), mpq.absmax(wd, mode)
        xp = mpq.encode_nchw(xd, sa_d, a_bits, mpq.ACT_HRELU)
        wp, taps = mpq.encode_oihw(wd, sw_d, w_bits, mode)
        yi = torch.full(acc_ref.shape, -5, dtype=torch.int32, device=cuda)
        yf = torch.full(acc_ref.shape, float("nan"), dtype=torch.float32, device=cuda)
        mpq.conv(xp, a_bits, N, C, H, W, wp, w_bits, taps, O, 1, 1, stride, 0, yi, yf, sa_d, sw_d, mode)
        assert np.array_equal(yi.cpu().numpy(), acc_ref)
        assert rel_close(yf.cpu().numpy(), out_ref)
        out_max = torch.zeros(1, dtype=torch.float32, device=cuda)
        yf.fill_(float("nan"))
        mpq.conv_fused(xp, a_bits, N, C, H, W, wp, w_bits, taps, O, 1, 1, stride, 0, None, yf, sa_d, sw_d, mode,
                       _dev(res, cuda), True, out_max)
        got = yf.cpu().numpy()
        assert rel_close(got, want)
        assert float(out_max.item()) == float(got.max())


@pytest.mark.parametrize("stride,pad", [(1, 1), (2, 1), (1, 0), (2, 0)])
@pytest.mark.parametrize("a_bits,w_bits", [(4, 4), (1, 8), (3, 2), (2, 5), (5, 4)])
def test_conv3x3_over_64_channels(mpq, cuda, a_bits, w_bits, stride, pad):
    """3 x 3 convolutions over 64 channels (the first stage of a residual stack): with activations of up to
    4 bits one thread keeps the whole window of its output pixel in registers; 5 bits take the tiled kernel.
    Small images (every pixel on the border at 3 x 4), ragged pixel and channel counts, both outputs,
    residual + max(., 0) + the next encoder's range in the store."""
    for (N, H, W, O) in ((2, 3, 4, 8), (3, 12, 9, 72)):
        if a_bits + w_bits > 8:
            O = min(O, 40)
        x = inputs.uniform_levels(25, 10 * stride + pad, (N, 64, H, W), a_bits)
        w = inputs.uniform_levels(25, 50 + O, (O, 64, 3, 3), w_bits) * np.float32(1.7)
        acc_ref, out_ref, s_a, s_w = oracle.conv_layer(x, w, a_bits, w_bits, stride, pad, True, oracle.HRELU)
        res = inputs.normal(25, 7, out_ref.shape)
        want = oracle.epilogue(out_ref, None, res, True)
        xd, wd = _dev(x, cuda), _dev(w, cuda)
        sa_d, sw_d = mpq.absmax(xd, 0, mpq.ACT_HRELU), mpq.absmax(wd, mpq.SCALE_PER_ROW)
        xp = mpq.encode_nchw(xd, sa_d, a_bits, mpq.ACT_HRELU)
        wp, taps = mpq.encode_oihw(wd, sw_d, w_bits, mpq.SCALE_PER_ROW)
        yi = torch.full(acc_ref.shape, -5, dtype=torch.int32, device=cuda)
        yf = torch.full(acc_ref.shape, float("nan"), dtype=torch.float32, device=cuda)
        mpq.conv(xp, a_bits, N, 64, H, W, wp, w_bits, taps, O, 3, 3, stride, pad, yi, yf, sa_d, sw_d, mpq.SCALE_PER_ROW)
        assert np.array_equal(yi.cpu().numpy(), acc_ref), (N, H, W, O)
        assert rel_close(yf.cpu().numpy(), out_ref), (N, H, W, O)
        out_max = torch.zeros(1, dtype=torch.float32, device=cuda)
        yf.fill_(float("nan"))
        mpq.conv_fused(xp, a_bits, N, 64, H, W, wp, w_bits, taps, O, 3, 3, stride, pad, None, yf, sa_d, sw_d,
                       mpq.SCALE_PER_ROW, _dev(res, cuda), True, out_max)
        got = yf.cpu().numpy()
        assert rel_close(got, want), (N, H, W, O)
        assert float(out_max.item()) == float(got.max())
