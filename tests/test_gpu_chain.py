"""GPU parity of the chained-layer entry points, through the C ABI, against the CPU oracle:
the trigonometric Encoder form, the fused GEMM store (bias, residual, max), including the shapes that
run with k-groups inside the CTA, the convolution that runs its consumer's Encoder in the store, and the
host entry point with resident weights.  int32 and packed planes bit-exact, fp32 within 1e-5
relative (exact at 0)."""
import numpy as np
import pytest
import torch

import oracle
from paper_1905_13389_b200 import inputs
from tests._util import rel_close, unpack_planes

pytestmark = pytest.mark.gpu


def _dev(a, cuda):
    return torch.from_numpy(np.ascontiguousarray(a)).to(cuda)


# ---------------------------------------------------------------------------- trigonometric encoder
@pytest.mark.parametrize("bits", range(1, 9))
@pytest.mark.parametrize("shape", [(1, 1), (3, 33), (5, 1000), (2, 1024), (4, 2500)])
def test_trig_encoder_matches_the_oracle(mpq, cuda, bits, shape):
    """Eq. 11's sine encoders (and their family at other widths) against the oracle's own sine route:
    both form each argument with one fp32 multiply, so the planes agree bit for bit -- ties, values a
    rounding away from every level boundary, NaN, infinities and out-of-range inputs included."""
    rng = np.random.default_rng(bits * 31 + shape[1])
    x = (rng.standard_normal(shape) * 0.8).astype(np.float32)
    x.flat[::5] = 0.0
    L = 2 ** bits - 1
    edges = np.array([(2 * n - L - 1) / L for n in range(0, L + 2)], dtype=np.float32)
    near = np.concatenate([edges, np.nextafter(edges, np.float32(9)), np.nextafter(edges, np.float32(-9))])
    flat = x.reshape(-1)
    m = min(flat.size, near.size)
    flat[:m] = near[:m]
    if flat.size > 800:
        flat[700:705] = [np.nan, np.inf, -np.inf, 1e30, -1e30]
    xd = _dev(x, cuda)
    for act in (mpq.ACT_HTANH, mpq.ACT_HRELU):
        for per_row in (False, True):
            s = rng.uniform(0.5, 1.5, shape[0]).astype(np.float32) if per_row else np.ones(1, np.float32)
            planes = mpq.encode_with(mpq.ENC_TRIG, xd, _dev(s, cuda), bits, int(per_row), act)
            u = unpack_planes(planes.cpu().numpy(), shape[1])
            ref = oracle.levels(oracle.quantize_trig(x, s, bits, per_row=per_row, act=act), bits)
            assert np.array_equal(u, ref)


def test_trig_encoder_and_level_encoder_agree_away_from_boundaries(mpq, cuda):
    """The two Encoder forms spell the same planes for inputs that are not within a rounding of a
    level boundary (there each takes its own decision); range 1 with exact level centres and ties."""
    one = _dev(np.ones(1, np.float32), cuda)
    for bits in (1, 2, 3, 5, 8):
        x = inputs.uniform_levels(11, bits, (9, 777), bits)
        x[0, :7] = 0.0
        xd = _dev(x, cuda)
        a = mpq.encode_with(mpq.ENC_TRIG, xd, one, bits).cpu().numpy()
        b = mpq.encode_with(mpq.ENC_LEVELS, xd, one, bits).cpu().numpy()
        c = mpq.encode(xd, one, bits).cpu().numpy()
        assert np.array_equal(a, b) and np.array_equal(b, c)
    t2 = np.array([[-1.0, -1.0 / 3.0, 1.0 / 3.0, 1.0]], dtype=np.float32)          # Table 2's four levels
    u = unpack_planes(mpq.encode_with(mpq.ENC_TRIG, _dev(t2, cuda), one, 2).cpu().numpy(), 4)
    assert u.tolist() == [[0, 1, 2, 3]]
    rc = mpq.lib().mpq_encode_with(7, 1, 1, 1, 1, 1, 0, 0, 2, 16, None)
    assert rc == 3                                                                  # unknown encoder form


# ----------------------------------------------------------------------------------- fused GEMM store
def _fused_case(mpq, cuda, x, w, a_bits, w_bits, per_row, a_act, outs, glue):
    m, k = x.shape
    n = w.shape[0]
    acc_ref, out_ref, s_a, s_w = oracle.linear(x, w, a_bits, w_bits, w_per_row=per_row, a_act=a_act)
    rng = np.random.default_rng(m + n + k)
    scale = float(np.abs(out_ref).max()) or 1.0
    bias = (rng.standard_normal(n) * 0.3 * scale).astype(np.float32) if glue else None
    res = (rng.standard_normal((m, n)) * 0.3 * scale).astype(np.float32) if glue else None
    ref = oracle.epilogue(out_ref, bias, res, relu=glue)
    xd, wd = _dev(x, cuda), _dev(w, cuda)
    sa_d, sw_d = mpq.absmax(xd, 0, a_act), mpq.absmax(wd, int(per_row))
    ap, wp = mpq.encode(xd, sa_d, a_bits, 0, a_act), mpq.encode(wd, sw_d, w_bits, int(per_row))
    ci = torch.full((m, n), -7, dtype=torch.int32, device=cuda) if "i" in outs else None
    cf = torch.full((m, n), float("nan"), dtype=torch.float32, device=cuda) if "f" in outs else None
    mpq.gemm_fused(ap, a_bits, wp, w_bits, m, n, k, ci, cf, sa_d, sw_d, int(per_row),
                   None if bias is None else _dev(bias, cuda), None if res is None else _dev(res, cuda), glue)
    if ci is not None:
        assert np.array_equal(ci.cpu().numpy(), acc_ref)
    if cf is not None:
        assert rel_close(cf.cpu().numpy(), ref)
        if glue:
            assert float(cf.min()) >= 0.0 and float((cf == 0).float().mean()) > 0.05


@pytest.mark.parametrize("m,n,k", [(64, 2048, 32768), (50, 1000, 20000), (17, 64, 9216), (128, 300, 2100), (4, 4, 64)])
@pytest.mark.parametrize("bits", [(2, 2), (1, 1), (3, 2), (4, 4), (8, 8)])
def test_gemm_fused_few_tiles_long_k(mpq, cuda, m, n, k, bits):
    """Few output tiles and a long k (the shapes whose CTAs are split into k-groups, and ragged ones
    beside them): results are the oracle's -- int32 only, fp32 only and both, with and without the
    glue in the store."""
    a_bits, w_bits = bits
    assert (2 ** a_bits - 1) * (2 ** w_bits - 1) * k < 2 ** 31
    x = inputs.uniform_levels(12, a_bits, (m, k), a_bits)
    w = inputs.uniform_levels(12, 10 + w_bits, (n, k), w_bits)
    for outs, glue in (("i", False), ("f", False), ("if", True), ("f", True)):
        _fused_case(mpq, cuda, x, w, a_bits, w_bits, True, mpq.ACT_HTANH, outs, glue)


def test_gemm_fused_many_tiles_and_config2(mpq, cuda):
    """A product of many tiles with the glue in its store, then the fully-connected layer of the
    workloads (64 x 4096 x 9216, W2A2, per-channel weight ranges)."""
    x = inputs.uniform_levels(12, 1, (70, 1200), 3)
    w = inputs.uniform_levels(12, 2, (333, 1200), 2)
    _fused_case(mpq, cuda, x, w, 3, 2, False, mpq.ACT_HRELU, "if", True)
    c = inputs.config2()
    _fused_case(mpq, cuda, c["x"], c["w"], 2, 2, True, mpq.ACT_HRELU, "f", False)
    _fused_case(mpq, cuda, c["x"], c["w"], 2, 2, True, mpq.ACT_HRELU, "if", True)


def test_gemm_fused_argument_checks(mpq, cuda):
    L = mpq.lib()
    a = torch.zeros(4096, dtype=torch.int32, device=cuda)
    f = torch.zeros(4096, dtype=torch.float32, device=cuda)
    # the glue needs the fp32 output
    assert L.mpq_gemm_fused(a.data_ptr(), 2, a.data_ptr(), 2, 4, 4, 32, a.data_ptr(), None, 4, None, None, 0,
                            f.data_ptr(), None, 0, None) == 1
    assert L.mpq_gemm_fused(a.data_ptr(), 2, a.data_ptr(), 2, 4, 4, 32, a.data_ptr(), None, 4, None, None, 0,
                            None, None, 1, None) == 1


# ------------------------------------------------------------- convolution with the consumer's encoder
def _pack_nhwc(u, bits):
    """Level indices [N][O][Ho][Wo] -> planes [bits][N][Ho][Wo][O/32] (test-side packer)."""
    N, O, Ho, Wo = u.shape
    t = u.transpose(0, 2, 3, 1).reshape(N, Ho, Wo, O // 32, 32).astype(np.uint64)
    weights = np.uint64(1) << np.arange(32, dtype=np.uint64)
    return np.stack([(((t >> np.uint64(p)) & np.uint64(1)) * weights).sum(axis=4).astype(np.uint32) for p in range(bits)])


@pytest.mark.parametrize("w_bits,O", [(1, 160), (2, 96), (4, 64), (3, 32), (6, 64), (8, 32)])
@pytest.mark.parametrize("C,ksz,stride,pad", [(64, 3, 1, 1), (128, 1, 2, 0), (32, 3, 2, 1)])
def test_conv_encoded_writes_the_consumers_planes(mpq, cuda, w_bits, O, C, ksz, stride, pad):
    """The consumer's Encoder in the store: planes equal the oracle's codes of the oracle's fp32 output
    (range given beforehand), for every tile height of the kernel (16, 32, 64, 128 channels), with and
    without the fp32 store, residual and max; the fp32 output and the accumulators stay the oracle's."""
    rng = np.random.default_rng(w_bits * 100 + O + C)
    a_bits, next_bits = 3, 4
    x = inputs.uniform_levels(13, C + ksz, (2, C, 9, 7), a_bits)
    w = rng.standard_normal((O, C, ksz, ksz)).astype(np.float32)
    acc_ref, out_ref, s_a, s_w = oracle.conv_layer(x, w, a_bits, w_bits, stride, pad, True, oracle.HTANH)
    res = (rng.standard_normal(out_ref.shape) * 0.4 * np.abs(out_ref).max()).astype(np.float32)
    xd, wd = _dev(x, cuda), _dev(w, cuda)
    sa_d, sw_d = mpq.absmax(xd), mpq.absmax(wd, mpq.SCALE_PER_ROW)
    xp = mpq.encode_nchw(xd, sa_d, a_bits)
    wp, taps = mpq.encode_oihw(wd, sw_d, w_bits, mpq.SCALE_PER_ROW)
    N, _, H, W = x.shape
    for residual, relu, keep_f32, act in ((None, False, True, mpq.ACT_HTANH), (res, True, True, mpq.ACT_HRELU),
                                          (res, False, False, mpq.ACT_HRELU), (None, True, False, mpq.ACT_HTANH)):
        ref = oracle.epilogue(out_ref, None, residual, relu)
        s_next = np.array([0.6 * np.abs(ref).max()], np.float32)          # a range fixed beforehand; part of the data clips
        q_next = oracle.quantize(ref, s_next, next_bits, act=act)
        want = _pack_nhwc(oracle.levels(q_next, next_bits), next_bits)
        yi = torch.full(acc_ref.shape, -7, dtype=torch.int32, device=cuda)
        yf = torch.full(acc_ref.shape, float("nan"), dtype=torch.float32, device=cuda) if keep_f32 else None
        guard = 64
        whole = torch.full((want.size + 2 * guard,), 0x5A5A5A5A, dtype=torch.int32, device=cuda)
        planes = whole[guard:guard + want.size].view(*want.shape)
        mpq.conv_encoded(xp, a_bits, N, C, H, W, wp, w_bits, taps, O, ksz, ksz, stride, pad, yi, yf, sa_d, sw_d,
                         mpq.SCALE_PER_ROW, None if residual is None else _dev(residual, cuda), relu, None,
                         _dev(s_next, cuda), act, next_bits, planes)
        assert np.array_equal(planes.cpu().numpy().view(np.uint32), want)
        hw = whole.cpu().numpy()
        assert np.all(hw[:guard] == 0x5A5A5A5A) and np.all(hw[guard + want.size:] == 0x5A5A5A5A)
        assert np.array_equal(yi.cpu().numpy(), acc_ref)
        if keep_f32:
            assert np.array_equal(yf.cpu().numpy(), ref)
        assert len(np.unique(oracle.levels(q_next, next_bits))) > 4


def test_conv_encoded_feeds_the_next_convolution(mpq, cuda):
    """Two chained layers with a fixed HReLU range between them: conv1 writes conv2's planes from its
    store; conv2 on those planes equals the oracle's conv2 on the oracle's quantized conv1 output."""
    rng = np.random.default_rng(5)
    x = inputs.uniform_levels(13, 1, (2, 64, 10, 10), 4)
    w1 = rng.standard_normal((64, 64, 3, 3)).astype(np.float32)
    w2 = rng.standard_normal((32, 64, 3, 3)).astype(np.float32)
    acc1, out1, s_a, s_w1 = oracle.conv_layer(x, w1, 4, 4, 1, 1, True, oracle.HTANH)
    mid = oracle.epilogue(out1, None, None, True)
    s_mid = np.array([0.5 * mid.max()], np.float32)
    q_mid = oracle.quantize(mid, s_mid, 4, act=oracle.HRELU)
    s_w2 = oracle.absmax(w2, per_row=True)
    acc2 = oracle.conv(q_mid, oracle.quantize(w2, s_w2, 4, per_row=True), 1, 1)
    out2 = oracle.scale(acc2, s_mid[0], s_w2, 4, 4)
    xd = _dev(x, cuda)
    sa_d = mpq.absmax(xd)
    xp = mpq.encode_nchw(xd, sa_d, 4)
    w1d, w2d = _dev(w1, cuda), _dev(w2, cuda)
    sw1, sw2 = mpq.absmax(w1d, 1), mpq.absmax(w2d, 1)
    wp1, t1 = mpq.encode_oihw(w1d, sw1, 4, 1)
    wp2, t2 = mpq.encode_oihw(w2d, sw2, 4, 1)
    smid_d = _dev(s_mid, cuda)
    mid_planes = mpq.conv_encoded(xp, 4, 2, 64, 10, 10, wp1, 4, t1, 64, 3, 3, 1, 1, None, None, sa_d, sw1, 1,
                                  None, True, None, smid_d, mpq.ACT_HRELU, 4)
    yi = torch.empty(acc2.shape, dtype=torch.int32, device=cuda)
    yf = torch.empty(acc2.shape, dtype=torch.float32, device=cuda)
    mpq.conv(mid_planes, 4, 2, 64, 10, 10, wp2, 4, t2, 32, 3, 3, 1, 1, yi, yf, smid_d, sw2, 1)
    assert np.array_equal(yi.cpu().numpy(), acc2)
    assert rel_close(yf.cpu().numpy(), out2)


def test_conv_encoded_argument_checks(mpq, cuda):
    L = mpq.lib()
    a = torch.zeros(1 << 16, dtype=torch.int32, device=cuda)
    f = torch.zeros(1 << 16, dtype=torch.float32, device=cuda)
    def call(O=32, next_bits=4, next_act=1, next_scale=f.data_ptr(), planes=a.data_ptr()):
        return L.mpq_conv_encoded(a.data_ptr(), 2, 1, 64, 8, 8, a.data_ptr(), 2, a.data_ptr(), O, 3, 3, 1, 1,
                                  None, None, f.data_ptr(), f.data_ptr(), 0, None, 0, None,
                                  next_scale, next_act, next_bits, planes, None)
    assert call(O=40) == 3 and call(next_bits=9) == 3 and call(next_act=5) == 3
    assert call(next_scale=None) == 1
    assert call(planes=a.data_ptr() + 4) == 5
    assert call(planes=None) == 1                      # nothing at all to write


# ------------------------------------------------------------------ host entry point, resident weights
@pytest.mark.parametrize("m,n,k,per_row", [(64, 96, 512, False), (1500, 200, 1000, True)])
def test_linear_host_prepared(mpq, cuda, m, n, k, per_row):
    x = inputs.uniform_levels(14, 1, (m, k), 3)
    w = inputs.uniform_levels(14, 2, (n, k), 4)
    acc_ref, out_ref, _, _ = oracle.linear(x, w, 3, 4, w_per_row=per_row, a_act=oracle.HRELU)
    wd = _dev(w, cuda)
    sw = mpq.absmax(wd, int(per_row))
    wp = mpq.encode(wd, sw, 4, int(per_row))                        # once, "offline"
    xh = torch.from_numpy(x).pin_memory()
    oi = torch.full((m, n), -7, dtype=torch.int32).pin_memory()
    of = torch.full((m, n), float("nan"), dtype=torch.float32).pin_memory()
    for _ in range(2):
        mpq.linear_host_prepared(xh, wp, sw, n, 3, 4, mpq.ACT_HRELU, int(per_row), oi, of)
        assert np.array_equal(oi.numpy(), acc_ref)
        assert rel_close(of.numpy(), out_ref)
    need = mpq.linear_host_prepared_workspace(m, n, k, 3)
    small = torch.empty(need - 256, dtype=torch.uint8, device=cuda)
    rc = mpq.lib().mpq_linear_host_prepared(xh.data_ptr(), wp.data_ptr(), sw.data_ptr(), m, n, k, 3, 4, 1, int(per_row),
                                            oi.data_ptr(), None, small.data_ptr(), small.numel(), None)
    assert rc == 7


# -------------------------------------------------------------- per-row range + encode in one pass
@pytest.mark.parametrize("bits", [1, 2, 4, 8])
@pytest.mark.parametrize("shape", [(1, 1), (5, 33), (7, 1000), (3, 1024), (6, 2500), (4, 9216), (2, 49152), (2, 50000)])
def test_encode_ranged_equals_range_then_encode(mpq, cuda, bits, shape):
    """One pass over memory gives the oracle's per-row ranges and the oracle's codes under those ranges
    (NaN ignored by the range and sent to the level above zero; ties, infinities beyond the range; rows
    longer than the staging buffer take the two-pass route with the same results)."""
    rng = np.random.default_rng(bits * 1000 + shape[1])
    x = (rng.standard_normal(shape) * rng.uniform(0.01, 3.0, size=(shape[0], 1))).astype(np.float32)
    x.flat[::9] = 0.0
    if shape[1] > 40:
        x[0, 5] = np.nan
        x[-1, 7] = -1e30
    xd = _dev(x, cuda)
    for act in (mpq.ACT_HTANH, mpq.ACT_HRELU):
        s_ref = oracle.absmax(x, True, act)
        scale, planes = mpq.encode_ranged(xd, bits, act)
        assert np.array_equal(scale.cpu().numpy(), s_ref)
        u = unpack_planes(planes.cpu().numpy(), shape[1])
        assert np.array_equal(u, oracle.levels(oracle.quantize(x, s_ref, bits, per_row=True, act=act), bits))
    # an all-zero row has range 0: every code is the level above zero
    z = torch.zeros((2, 300), dtype=torch.float32, device=cuda)
    scale, planes = mpq.encode_ranged(z, bits)
    assert float(scale.abs().max()) == 0.0
    assert np.all(unpack_planes(planes.cpu().numpy(), 300) == 2 ** (bits - 1))
