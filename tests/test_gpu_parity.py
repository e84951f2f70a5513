"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded inputs.  int32 results must be bit-exact; fp32 results within 1e-5 relative (exact at 0)."""
import numpy as np
import pytest
import torch

import oracle
from paper_1905_13389_b200 import inputs
from tests._util import pack_levels, rel_close, unpack_planes

pytestmark = pytest.mark.gpu

CANARY = np.int32(0x5A5A5A5A)


def _dev(a, cuda):
    return torch.from_numpy(np.ascontiguousarray(a)).to(cuda)


def _guarded(shape, dtype, cuda, guard=64):
    """Flat buffer with canary words on both sides of the payload; returns (payload view, whole)."""
    n = int(np.prod(shape))
    whole = torch.full((n + 2 * guard,), int(CANARY), dtype=torch.int32, device=cuda)
    payload = whole[guard:guard + n].view(dtype).view(*shape) if dtype != torch.int32 else whole[guard:guard + n].view(*shape)
    return payload, whole


def _canaries_intact(whole, n, guard=64):
    w = whole.cpu().numpy()
    return bool(np.all(w[:guard] == CANARY) and np.all(w[guard + n:] == CANARY))


# ------------------------------------------------------------------------------------------ range
@pytest.mark.parametrize("shape", [(1, 1), (3, 1000), (64, 512), (5, 8192 + 37), (129, 4099)])
def test_absmax(mpq, cuda, shape):
    rng = np.random.default_rng(shape[1])
    x = rng.standard_normal(shape).astype(np.float32)
    x[0, 0] = np.nan
    xd = _dev(x, cuda)
    for act in (mpq.ACT_HTANH, mpq.ACT_HRELU):
        got = mpq.absmax(xd, mpq.SCALE_PER_TENSOR, act).cpu().numpy()
        assert np.array_equal(got, oracle.absmax(x, False, act))
        got = mpq.absmax(xd, mpq.SCALE_PER_ROW, act).cpu().numpy()
        assert np.array_equal(got, oracle.absmax(x, True, act))


def test_absmax_unaligned_view(mpq, cuda):
    """Row stride not a multiple of 4 elements: the scalar path."""
    rng = np.random.default_rng(5)
    x = rng.standard_normal((7, 1001)).astype(np.float32)
    got = mpq.absmax(_dev(x, cuda), mpq.SCALE_PER_ROW).cpu().numpy()
    assert np.array_equal(got, np.abs(x).max(axis=1))


# ---------------------------------------------------------------------------------------- encoder
@pytest.mark.parametrize("bits", range(1, 9))
@pytest.mark.parametrize("shape", [(1, 1), (2, 31), (3, 32), (5, 33), (4, 1000), (3, 1024), (2, 1025), (9, 2500)])
def test_encode_rows_codes(mpq, cuda, bits, shape):
    rng = np.random.default_rng(bits * 100 + shape[1])
    x = (rng.standard_normal(shape) * 0.7).astype(np.float32)
    x.flat[:: 7] = 0.0                                    # exact ties
    xd = _dev(x, cuda)
    for act in (mpq.ACT_HTANH, mpq.ACT_HRELU):
        for per_row in (False, True):
            s = oracle.absmax(x, per_row, act)
            planes, whole = _guarded((bits, shape[0], mpq.row_words(shape[1])), torch.int32, cuda)
            mpq.encode(xd, _dev(s, cuda), bits, int(per_row), act, out=planes)
            u = unpack_planes(planes.cpu().numpy(), shape[1])
            q = oracle.quantize(x, s, bits, per_row=per_row, act=act)
            assert np.array_equal(u, oracle.levels(q, bits))
            assert _canaries_intact(whole, planes.numel())


def test_encode_rows_uniform_levels_and_table2(mpq, cuda):
    """All levels exercised (range 1), including the four printed levels of Table 2."""
    one = _dev(np.ones(1, np.float32), cuda)
    t2 = np.array([[-1.0, -1.0 / 3.0, 1.0 / 3.0, 1.0]], dtype=np.float32)
    u = unpack_planes(mpq.encode(_dev(t2, cuda), one, 2).cpu().numpy(), 4)
    assert u.tolist() == [[0, 1, 2, 3]]
    for bits in (1, 2, 3, 5, 8):
        x = inputs.uniform_levels(9, bits, (17, 777), bits)
        u = unpack_planes(mpq.encode(_dev(x, cuda), one, bits).cpu().numpy(), 777)
        assert np.array_equal(u, oracle.levels(oracle.quantize(x, 1.0, bits), bits))
        assert set(np.unique(u).tolist()) == set(range(2 ** bits))


def test_encode_degenerate_scale(mpq, cuda):
    x = _dev(np.array([[-3.0, -0.1, 0.0, 0.1, 3.0, np.nan]], np.float32), cuda)
    for s in (0.0, -1.0, np.inf, np.nan):
        u = unpack_planes(mpq.encode(x, _dev(np.array([s], np.float32), cuda), 3).cpu().numpy(), 6)
        assert u.tolist() == [[4] * 6]                    # q = +1 everywhere


@pytest.mark.parametrize("act", [0, 1])
def test_encode_subnormal_scale_with_zeros(mpq, cuda, act):
    """A positive subnormal range makes 1/s overflow to infinity, so an exact zero gives 0 * inf = NaN
    and must land on the level above zero on every path: full 1024-element rows (lane-local path),
    a ragged row (ballot path) and the NCHW encoder."""
    rng = np.random.default_rng(40)
    s = np.array([1e-40], np.float32)
    assert 0.0 < float(s[0]) < 2.9e-39
    for shape in ((3, 1024), (2, 777)):
        x = (rng.standard_normal(shape) * 1e-39).astype(np.float32)
        x[:, ::5] = 0.0
        u = unpack_planes(mpq.encode(_dev(x, cuda), _dev(s, cuda), 3, 0, act).cpu().numpy(), shape[1])
        assert np.array_equal(u, oracle.levels(oracle.quantize(x, s, 3, act=act), 3))
    xn = (rng.standard_normal((2, 32, 5, 7)) * 1e-39).astype(np.float32)
    xn[:, ::3] = 0.0
    planes = mpq.encode_nchw(_dev(xn, cuda), _dev(s, cuda), 3, act).cpu().numpy()      # [bits][N][H][W][1]
    u = unpack_planes(planes.reshape(3, -1, 1), 32).reshape(2, 5, 7, 32).transpose(0, 3, 1, 2)
    assert np.array_equal(u, oracle.levels(oracle.quantize(xn, s, 3, act=act), 3))


@pytest.mark.parametrize("bits", [1, 2, 4, 7])
def test_encode_rows_full_segments_with_specials(mpq, cuda, bits):
    """Full 1024-element segments (the lean path) holding NaN, +-inf, exact ties, values far
    outside the range and values one ulp either side of every level boundary."""
    rng = np.random.default_rng(bits)
    rows, k = 6, 3 * 1024 + 100
    x = (rng.standard_normal((rows, k)) * 0.6).astype(np.float32)
    L = 2 ** bits - 1
    edges = np.array([(2 * n - L - 1) / L for n in range(0, L + 2)], dtype=np.float32)   # level boundaries
    near = np.concatenate([edges, np.nextafter(edges, np.float32(9)), np.nextafter(edges, np.float32(-9))])
    x[0, : near.size] = near
    x[1, 5] = np.nan; x[1, 1500] = np.nan; x[2, 2047] = np.inf; x[2, 2048] = -np.inf
    x[3, ::3] = 0.0; x[4, 10] = 1e30; x[4, 11] = -1e30; x[5, 7] = np.float32(1e-42); x[5, 8] = np.float32(-1e-42)
    xd = _dev(x, cuda)
    for act in (mpq.ACT_HTANH, mpq.ACT_HRELU):
        for s in (np.ones(1, np.float32), np.array([0.37], np.float32), np.array([np.nan], np.float32)):
            planes = mpq.encode(xd, _dev(s, cuda), bits, 0, act)
            u = unpack_planes(planes.cpu().numpy(), k)
            assert np.array_equal(u, oracle.levels(oracle.quantize(x, s, bits, act=act), bits))


@pytest.mark.parametrize("bits,act", [(2, 0), (3, 1), (8, 0)])
def test_encode_every_float_of_a_binade(mpq, cuda, bits, act):
    """Every float32 with |x| in [1/2, 1) -- 16.8 million inputs, all level boundaries of the upper half
    of the range with their neighbours -- against the oracle's quantizer, plane by plane.  (The same
    comparison over all 2^32 bit patterns was run once when the FMA-pipe quantizer was written.)"""
    lo, hi = np.float32(0.5).view(np.uint32), np.float32(1.0).view(np.uint32)
    pos = np.arange(lo, hi, dtype=np.uint32)
    k = 1 << 20
    x = np.concatenate([pos, pos | np.uint32(0x80000000)]).view(np.float32).reshape(-1, k)
    one = _dev(np.ones(1, np.float32), cuda)
    planes = mpq.encode(_dev(x, cuda), one, bits, 0, act).cpu().numpy().view(np.uint32)
    u = oracle.levels(oracle.quantize(x, 1.0, bits, act=act), bits)
    for p in range(bits):
        ref = np.packbits(((u >> p) & 1).astype(np.uint8), axis=1, bitorder="little").view(np.uint32)
        assert np.array_equal(ref, planes[p]), p


def test_encode_nchw_every_float_of_a_binade(mpq, cuda):
    """The same 16.8 million inputs through the NCHW encoder (4 bits, HReLU), word by word."""
    lo, hi = np.float32(0.5).view(np.uint32), np.float32(1.0).view(np.uint32)
    pos = np.arange(lo, hi, dtype=np.uint32)
    x = np.concatenate([pos, pos | np.uint32(0x80000000)]).view(np.float32).reshape(16, 64, 128, 128)
    one = _dev(np.ones(1, np.float32), cuda)
    planes = mpq.encode_nchw(_dev(x, cuda), one, 4, mpq.ACT_HRELU).cpu().numpy().view(np.uint32)   # [4][N][H][W][2]
    u = oracle.levels(oracle.quantize(x, 1.0, 4, act=oracle.HRELU), 4).transpose(0, 2, 3, 1)       # [N][H][W][C]
    for p in range(4):
        ref = np.packbits(((u >> p) & 1).astype(np.uint8), axis=3, bitorder="little").view(np.uint32)
        assert np.array_equal(ref.reshape(planes[p].shape), planes[p]), p


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
@pytest.mark.parametrize("shape", [(2, 32, 5, 7), (1, 64, 9, 9), (3, 128, 4, 6), (2, 256, 14, 14)])
def test_encode_nchw_codes(mpq, cuda, bits, shape):
    rng = np.random.default_rng(bits + shape[1])
    x = rng.standard_normal(shape).astype(np.float32)
    N, C, H, W = shape
    x[0, 3, 1, 2] = np.nan; x[0, 5, 0, 0] = np.inf; x[0, 6, 0, 0] = -np.inf; x[:, 7] = 0.0
    for act in (mpq.ACT_HTANH, mpq.ACT_HRELU):
        s = oracle.absmax(x, False, act)
        if not np.isfinite(s[0]):
            s = np.ones(1, np.float32)
        planes = mpq.encode_nchw(_dev(x, cuda), _dev(s, cuda), bits, act).cpu().numpy()
        u = unpack_planes(planes.reshape(bits, N * H * W, C // 32), C).reshape(N, H, W, C).transpose(0, 3, 1, 2)
        assert np.array_equal(u, oracle.levels(oracle.quantize(x, s, bits, act=act), bits))


@pytest.mark.parametrize("shape", [(5, 32, 3, 3), (16, 64, 3, 3), (7, 128, 1, 1), (20, 64, 1, 1)])
def test_encode_oihw_codes_and_tap_sums(mpq, cuda, shape):
    rng = np.random.default_rng(shape[0])
    w = rng.standard_normal(shape).astype(np.float32)
    O, C, KH, KW = shape
    for bits in (1, 3, 8):
        for per_row in (False, True):
            s = oracle.absmax(w, per_row)
            planes, taps = mpq.encode_oihw(_dev(w, cuda), _dev(s, cuda), bits, int(per_row))
            q = oracle.quantize(w, s, bits, per_row=per_row)
            u = unpack_planes(planes.cpu().numpy(), KH * KW * C).reshape(O, KH, KW, C).transpose(0, 3, 1, 2)
            assert np.array_equal(u, oracle.levels(q, bits))
            ref_taps = q.astype(np.int64).sum(axis=1).reshape(O, KH * KW).T
            assert np.array_equal(taps.cpu().numpy(), ref_taps)


# ------------------------------------------------------------------------------------------- GEMM
def _gemm_case(mpq, cuda, x, w, a_bits, w_bits, w_per_row, a_act=0, both=True):
    m, k = x.shape
    n = w.shape[0]
    acc_ref, out_ref, s_a, s_w = oracle.linear(x, w, a_bits, w_bits, w_per_row=w_per_row, a_act=a_act)
    sa_d = mpq.absmax(_dev(x, cuda), mpq.SCALE_PER_TENSOR, a_act)
    sw_d = mpq.absmax(_dev(w, cuda), int(w_per_row))
    assert np.array_equal(sa_d.cpu().numpy(), s_a) and np.array_equal(sw_d.cpu().numpy(), s_w)
    ap = mpq.encode(_dev(x, cuda), sa_d, a_bits, mpq.SCALE_PER_TENSOR, a_act)
    wp = mpq.encode(_dev(w, cuda), sw_d, w_bits, int(w_per_row))
    ci, ci_whole = _guarded((m, n), torch.int32, cuda)
    cf, cf_whole = _guarded((m, n), torch.float32, cuda)
    mpq.gemm(ap, a_bits, wp, w_bits, m, n, k, ci if both else None, cf, sa_d, sw_d, int(w_per_row))
    if both:
        assert np.array_equal(ci.cpu().numpy(), acc_ref)
        assert _canaries_intact(ci_whole, m * n)
    assert rel_close(cf.cpu().numpy(), out_ref)
    assert _canaries_intact(cf_whole, m * n)
    return acc_ref


def test_gemm_config1(mpq, cuda):
    c = inputs.config1()
    acc = _gemm_case(mpq, cuda, c["x"], c["w"], c["a_bits"], c["w_bits"], c["w_per_row"])
    assert acc.shape == (64, 64)


@pytest.mark.parametrize("a_bits", range(1, 9))
@pytest.mark.parametrize("w_bits", range(1, 9))
def test_gemm_all_64_pairs_uniform_codes(mpq, cuda, a_bits, w_bits):
    """Every encoding choice, all levels present, ragged m / n / k (several tiles plus tails)."""
    m, n, k = 37, 150, 333
    x = inputs.uniform_levels(8, a_bits, (m, k), a_bits)
    w = inputs.uniform_levels(8, 10 + w_bits, (n, k), w_bits)
    _gemm_case(mpq, cuda, x, w, a_bits, w_bits, w_per_row=True)


@pytest.mark.parametrize("m,n,k", [(1, 1, 1), (1, 5, 32), (16, 16, 128), (130, 260, 1000), (300, 129, 4097), (64, 2000, 96)])
@pytest.mark.parametrize("bits", [(2, 2), (3, 3), (4, 4), (1, 2), (8, 8)])
def test_gemm_shapes(mpq, cuda, m, n, k, bits):
    a_bits, w_bits = bits
    rng = np.random.default_rng(m * 7 + n * 3 + k)
    x = np.maximum(rng.standard_normal((m, k)), 0).astype(np.float32)
    w = rng.standard_normal((n, k)).astype(np.float32)
    _gemm_case(mpq, cuda, x, w, a_bits, w_bits, w_per_row=False)


def test_gemm_hrelu_one_bit_closed_form(mpq, cuda):
    """1-bit activations after HReLU are all +1: every output row equals the weight-code row sums."""
    rng = np.random.default_rng(77)
    x = rng.standard_normal((9, 500)).astype(np.float32)
    w = rng.standard_normal((40, 500)).astype(np.float32)
    acc = _gemm_case(mpq, cuda, x, w, 1, 3, w_per_row=False, a_act=1)
    qw = oracle.quantize(w, oracle.absmax(w), 3).astype(np.int64)
    assert np.array_equal(acc, np.broadcast_to(qw.sum(axis=1), (9, 40)))


@pytest.mark.parametrize("a_bits,w_bits,k", [(8, 8, 33025), (4, 4, 100000), (1, 1, 300000)])
def test_gemm_extreme_codes_int32_headroom(mpq, cuda, a_bits, w_bits, k):
    """All-extreme codes at (or near) the largest k the int32 contract allows."""
    La, Lw = 2 ** a_bits - 1, 2 ** w_bits - 1
    ua = np.zeros((3, k), dtype=np.int64); ua[0] = La; ua[2, ::2] = La
    ub = np.zeros((2, k), dtype=np.int64); ub[1] = Lw
    rw = mpq.row_words(k)
    ap = _dev(pack_levels(ua, a_bits, rw).view(np.int32), cuda)
    bp = _dev(pack_levels(ub, w_bits, rw).view(np.int32), cuda)
    ci = torch.empty((3, 2), dtype=torch.int32, device=cuda)
    mpq.gemm(ap, a_bits, bp, w_bits, 3, 2, k, ci, None)
    ref = oracle.gemm(2 * ua - La, 2 * ub - Lw)
    assert np.array_equal(ci.cpu().numpy(), ref)
    assert abs(int(ref[0, 1])) == k * La * Lw


@pytest.mark.parametrize("a_bits,w_bits", [(2, 2), (4, 3), (7, 7)])
def test_gemm_equals_library_int8_product_of_decoded_integers(mpq, cuda, a_bits, w_bits):
    """Eq. 7-10 as a whole: the branch-decomposed product on bit-planes equals the plain integer
    product of the decoded odd integers, here computed by a library int8 GEMM on the device
    (an independent route; the integers come from the CPU oracle's quantizer)."""
    if not hasattr(torch, "_int_mm"):
        pytest.skip("no library int8 GEMM in this torch")
    m, n, k = 64, 96, 256
    x = inputs.uniform_levels(9, 40 + a_bits, (m, k), a_bits)
    w = inputs.uniform_levels(9, 50 + w_bits, (n, k), w_bits)
    one = _dev(np.ones(1, np.float32), cuda)
    qa = oracle.quantize(x, 1.0, a_bits).astype(np.int8)
    qb = oracle.quantize(w, 1.0, w_bits).astype(np.int8)
    ref = torch._int_mm(_dev(qa, cuda), _dev(np.ascontiguousarray(qb.T), cuda))
    ci = torch.empty((m, n), dtype=torch.int32, device=cuda)
    mpq.gemm(mpq.encode(_dev(x, cuda), one, a_bits), a_bits, mpq.encode(_dev(w, cuda), one, w_bits), w_bits,
             m, n, k, ci, None)
    assert torch.equal(ci, ref)
    assert np.array_equal(ci.cpu().numpy(), oracle.gemm(qa.astype(np.int16), qb.astype(np.int16)))


@pytest.mark.parametrize("pad_in,pad_out", [(4, 5), (1, 0), (0, 3)])
def test_strided_rows_through_the_c_abi(mpq, cuda, pad_in, pad_out):
    """Row strides larger than the row length (ldx > k for range and encode, ldc > n for the product),
    which the binding never passes: straight through the C entry points."""
    m, n, k = 21, 37, 2100
    rng = np.random.default_rng(pad_in * 7 + pad_out)
    xw = rng.standard_normal((m, k + pad_in)).astype(np.float32)
    ww = rng.standard_normal((n, k + pad_in)).astype(np.float32)
    xw[:, k:] = 1e9; ww[:, k:] = -1e9                      # poison outside the rows: must never be read as data
    x, w = np.ascontiguousarray(xw[:, :k]), np.ascontiguousarray(ww[:, :k])
    acc_ref, out_ref, s_a, s_w = oracle.linear(x, w, 3, 2, w_per_row=True)
    L = mpq.lib()
    xd, wd = _dev(xw, cuda), _dev(ww, cuda)
    sa = torch.empty(1, dtype=torch.float32, device=cuda)
    sw = torch.empty(n, dtype=torch.float32, device=cuda)
    st = torch.cuda.current_stream().cuda_stream
    assert L.mpq_absmax(xd.data_ptr(), m, k, k + pad_in, 0, 0, sa.data_ptr(), st) == 0
    assert L.mpq_absmax(wd.data_ptr(), n, k, k + pad_in, 1, 0, sw.data_ptr(), st) == 0
    assert np.array_equal(sa.cpu().numpy(), s_a) and np.array_equal(sw.cpu().numpy(), s_w)
    rw = mpq.row_words(k)
    ap = torch.empty((3, m, rw), dtype=torch.int32, device=cuda)
    wp = torch.empty((2, n, rw), dtype=torch.int32, device=cuda)
    assert L.mpq_encode(xd.data_ptr(), m, k, k + pad_in, sa.data_ptr(), 0, 0, 3, ap.data_ptr(), st) == 0
    assert L.mpq_encode(wd.data_ptr(), n, k, k + pad_in, sw.data_ptr(), 1, 0, 2, wp.data_ptr(), st) == 0
    ldc = n + pad_out
    ci = torch.full((m, ldc), 12345, dtype=torch.int32, device=cuda)
    cf = torch.full((m, ldc), 7.0, dtype=torch.float32, device=cuda)
    assert L.mpq_gemm(ap.data_ptr(), 3, wp.data_ptr(), 2, m, n, k, ci.data_ptr(), cf.data_ptr(), ldc,
                      sa.data_ptr(), sw.data_ptr(), 1, st) == 0
    assert np.array_equal(ci[:, :n].cpu().numpy(), acc_ref)
    assert rel_close(cf[:, :n].cpu().numpy(), out_ref)
    assert bool((ci[:, n:] == 12345).all()) and bool((cf[:, n:] == 7.0).all())     # the gap between rows is untouched


def test_gemm_config2_fc(mpq, cuda):
    c = inputs.config2()
    _gemm_case(mpq, cuda, c["x"], c["w"], 2, 2, w_per_row=True, both=False)


@pytest.mark.parametrize("w_bits,a_bits", inputs.SWEEP_BITS)
def test_gemm_config4_sampled_rows(mpq, cuda, w_bits, a_bits):
    """Full 4096^3 launch (the benchmark's configuration); the oracle checks 24 sampled rows x all
    columns, tile-boundary rows included, plus uniform-code operands so that every plane is live."""
    size = 4096
    for kind in ("gaussian", "uniform"):
        if kind == "gaussian":
            c = inputs.config4(w_bits, a_bits, size)
            x, w = c["x"], c["w"]
        else:
            x = inputs.uniform_levels(4, 100 + a_bits, (size, size), a_bits)
            w = inputs.uniform_levels(4, 200 + w_bits, (size, size), w_bits)
        s_a, s_w = oracle.absmax(x), oracle.absmax(w)
        xd, wd = _dev(x, cuda), _dev(w, cuda)
        sa_d, sw_d = mpq.absmax(xd), mpq.absmax(wd)
        assert np.array_equal(sa_d.cpu().numpy(), s_a) and np.array_equal(sw_d.cpu().numpy(), s_w)
        ap = mpq.encode(xd, sa_d, a_bits)
        wp = mpq.encode(wd, sw_d, w_bits)
        ci = torch.empty((size, size), dtype=torch.int32, device=cuda)
        cf = torch.empty((size, size), dtype=torch.float32, device=cuda)
        mpq.gemm(ap, a_bits, wp, w_bits, size, size, size, ci, cf, sa_d, sw_d)
        rows = sorted(set([0, 1, 15, 16, 63, 64, 127, 128, 2047, 2048, 4032, 4095] +
                          np.random.default_rng(a_bits * 8 + w_bits).integers(0, size, 12).tolist()))
        qa = oracle.quantize(x[rows], s_a, a_bits)
        qb = oracle.quantize(w, s_w, w_bits)
        acc_ref = oracle.gemm(qa, qb)
        got = ci[rows].cpu().numpy()
        assert np.array_equal(got, acc_ref)
        assert rel_close(cf[rows].cpu().numpy(), oracle.scale(acc_ref, s_a[0], s_w, a_bits, w_bits))
        if kind == "uniform" or a_bits > 1:
            assert np.unique(got).size > 16


# ------------------------------------------------------------------------------------------- conv
def _conv_case(mpq, cuda, x, w, a_bits, w_bits, stride, pad, w_per_channel=True, a_act=0):
    N, C, H, W = x.shape
    O, _, KH, KW = w.shape
    acc_ref, out_ref, s_a, s_w = oracle.conv_layer(x, w, a_bits, w_bits, stride, pad, w_per_channel, a_act)
    xd, wd = _dev(x, cuda), _dev(w, cuda)
    sa_d = mpq.absmax(xd, mpq.SCALE_PER_TENSOR, a_act)
    sw_d = mpq.absmax(wd, int(w_per_channel))
    xp = mpq.encode_nchw(xd, sa_d, a_bits, a_act)
    wp, taps = mpq.encode_oihw(wd, sw_d, w_bits, int(w_per_channel))
    yi, yi_whole = _guarded(acc_ref.shape, torch.int32, cuda)
    yf, yf_whole = _guarded(acc_ref.shape, torch.float32, cuda)
    mpq.conv(xp, a_bits, N, C, H, W, wp, w_bits, taps, O, KH, KW, stride, pad, yi, yf, sa_d, sw_d, int(w_per_channel))
    assert np.array_equal(yi.cpu().numpy(), acc_ref)
    assert rel_close(yf.cpu().numpy(), out_ref)
    assert _canaries_intact(yi_whole, acc_ref.size) and _canaries_intact(yf_whole, acc_ref.size)


@pytest.mark.parametrize("C", [32, 64, 128, 256])
@pytest.mark.parametrize("ksz,stride,pad", [(1, 1, 0), (1, 2, 0), (3, 1, 0), (3, 1, 1), (3, 2, 1)])
def test_conv_small(mpq, cuda, C, ksz, stride, pad):
    rng = np.random.default_rng(C + ksz * 10 + stride + pad)
    x = inputs.uniform_levels(7, C + ksz, (3, C, 9, 10), 3)
    w = rng.standard_normal((21, C, ksz, ksz)).astype(np.float32)
    _conv_case(mpq, cuda, x, w, 3, 2, stride, pad)


@pytest.mark.parametrize("a_bits,w_bits", [(1, 1), (2, 2), (4, 4), (8, 8), (2, 5), (6, 3)])
def test_conv_bit_pairs(mpq, cuda, a_bits, w_bits):
    x = inputs.uniform_levels(7, 50 + a_bits, (2, 64, 7, 7), a_bits)
    w = inputs.uniform_levels(7, 60 + w_bits, (40, 64, 3, 3), w_bits)
    _conv_case(mpq, cuda, x, w, a_bits, w_bits, 1, 1, w_per_channel=False)


def test_conv_config3(mpq, cuda):
    c = inputs.config3()
    _conv_case(mpq, cuda, c["x"], c["w"], 3, 3, 1, 1)


@pytest.mark.parametrize("C,ksz,stride,pad", [(64, 3, 1, 1), (128, 1, 2, 0), (32, 3, 2, 1)])
def test_conv_fused_store(mpq, cuda, C, ksz, stride, pad):
    """Residual add, max(.,0) and the running range folded into the store: same numbers as the
    separate steps (oracle convolution, one fp32 add, max), and the range equals their maximum."""
    rng = np.random.default_rng(C + ksz)
    x = inputs.uniform_levels(7, 70 + C, (3, C, 11, 9), 4)
    w = rng.standard_normal((40, C, ksz, ksz)).astype(np.float32)
    acc_ref, out_ref, s_a, s_w = oracle.conv_layer(x, w, 4, 3, stride, pad, True, oracle.HTANH)
    res = rng.standard_normal(out_ref.shape).astype(np.float32) * np.float32(0.5 * np.abs(out_ref).max())
    xd, wd = _dev(x, cuda), _dev(w, cuda)
    sa_d, sw_d = mpq.absmax(xd), mpq.absmax(wd, mpq.SCALE_PER_ROW)
    xp = mpq.encode_nchw(xd, sa_d, 4)
    wp, taps = mpq.encode_oihw(wd, sw_d, 3, mpq.SCALE_PER_ROW)
    N, _, H, W = x.shape
    yi = torch.empty(acc_ref.shape, dtype=torch.int32, device=cuda)
    for residual, relu in ((None, False), (res, False), (res, True), (None, True)):
        yf, yf_whole = _guarded(acc_ref.shape, torch.float32, cuda)
        seen = mpq.zero(torch.full((1,), 7.0, dtype=torch.float32, device=cuda))
        mpq.conv_fused(xp, 4, N, C, H, W, wp, 3, taps, 40, ksz, ksz, stride, pad, yi, yf, sa_d, sw_d,
                       mpq.SCALE_PER_ROW, None if residual is None else _dev(residual, cuda), relu, seen)
        ref = out_ref if residual is None else out_ref + residual
        if relu:
            ref = np.maximum(ref, np.float32(0))
        assert np.array_equal(yi.cpu().numpy(), acc_ref)
        assert np.array_equal(yf.cpu().numpy(), ref)                  # same single-rounded steps
        assert _canaries_intact(yf_whole, acc_ref.size)
        assert float(seen.cpu()[0]) == float(np.maximum(ref, 0).max())


def test_maxpool_range(mpq, cuda):
    x = np.random.default_rng(3).standard_normal((2, 5, 9, 12)).astype(np.float32)
    seen = mpq.zero(torch.ones(1, dtype=torch.float32, device=cuda))
    y = mpq.maxpool3x3s2(_dev(x, cuda), out_max=seen)
    ref = torch.nn.functional.max_pool2d(torch.from_numpy(x), 3, 2, 1).numpy()
    assert np.array_equal(y.cpu().numpy(), ref)
    assert float(seen.cpu()[0]) == float(np.maximum(ref, 0).max())


def test_conv_extreme_codes_int32_headroom(mpq, cuda):
    """All-extreme 8-bit codes at the largest channel count the int32 contract allows for a 3x3 filter
    (9 * 3584 * 255 * 255 = 2.10e9 < 2^31), with zero padding: interior outputs sit at -k L_a L_w and the
    border correction works on values whose staged form leaves the int32 range."""
    C, O = 3584, 3
    x = np.ones((1, C, 4, 4), np.float32)
    w = -np.ones((O, C, 3, 3), np.float32)
    w[1] = 1.0
    w[2, ::2] = 1.0
    acc_ref, out_ref, s_a, s_w = oracle.conv_layer(x, w, 8, 8, 1, 1, True, oracle.HTANH)
    assert int(acc_ref[0, 0, 1, 1]) == -9 * C * 255 * 255 and int(acc_ref[0, 1, 1, 1]) == 9 * C * 255 * 255
    xd, wd = _dev(x, cuda), _dev(w, cuda)
    sa_d, sw_d = mpq.absmax(xd), mpq.absmax(wd, mpq.SCALE_PER_ROW)
    xp = mpq.encode_nchw(xd, sa_d, 8)
    wp, taps = mpq.encode_oihw(wd, sw_d, 8, mpq.SCALE_PER_ROW)
    yi = torch.empty(acc_ref.shape, dtype=torch.int32, device=cuda)
    yf = torch.empty(acc_ref.shape, dtype=torch.float32, device=cuda)
    mpq.conv(xp, 8, 1, C, 4, 4, wp, 8, taps, O, 3, 3, 1, 1, yi, yf, sa_d, sw_d, mpq.SCALE_PER_ROW)
    assert np.array_equal(yi.cpu().numpy(), acc_ref)
    assert rel_close(yf.cpu().numpy(), out_ref)


def test_conv_1x1_equals_gemm(mpq, cuda):
    """A 1x1 stride-1 convolution is the GEMM of the pixel matrix with the weight matrix."""
    x = inputs.uniform_levels(7, 1, (2, 128, 6, 5), 4)
    w = inputs.uniform_levels(7, 2, (24, 128, 1, 1), 4)
    one = _dev(np.ones(1, np.float32), cuda)
    xp = mpq.encode_nchw(_dev(x, cuda), one, 4)
    wp, taps = mpq.encode_oihw(_dev(w, cuda), one, 4, mpq.SCALE_PER_TENSOR)
    yi = torch.empty((2, 24, 6, 5), dtype=torch.int32, device=cuda)
    mpq.conv(xp, 4, 2, 128, 6, 5, wp, 4, taps, 24, 1, 1, 1, 0, yi, None)
    rows = np.ascontiguousarray(x.transpose(0, 2, 3, 1).reshape(60, 128))
    ap = mpq.encode(_dev(rows, cuda), one, 4)
    bp = mpq.encode(_dev(w.reshape(24, 128), cuda), one, 4)
    ci = torch.empty((60, 24), dtype=torch.int32, device=cuda)
    mpq.gemm(ap, 4, bp, 4, 60, 24, 128, ci, None)
    assert np.array_equal(yi.cpu().numpy().transpose(0, 2, 3, 1).reshape(60, 24), ci.cpu().numpy())


# ---------------------------------------------------------------------------- whole-layer calls
@pytest.mark.parametrize("m,n,k,a_bits,w_bits,per_row", [(64, 64, 512, 2, 2, False), (33, 70, 1000, 3, 4, True)])
def test_linear_device(mpq, cuda, m, n, k, a_bits, w_bits, per_row):
    rng = np.random.default_rng(m + n)
    x = np.maximum(rng.standard_normal((m, k)), 0).astype(np.float32)
    w = rng.standard_normal((n, k)).astype(np.float32)
    oi = torch.empty((m, n), dtype=torch.int32, device=cuda)
    of = torch.empty((m, n), dtype=torch.float32, device=cuda)
    mpq.linear(_dev(x, cuda), _dev(w, cuda), a_bits, w_bits, mpq.ACT_HRELU, int(per_row), oi, of)
    acc_ref, out_ref, _, _ = oracle.linear(x, w, a_bits, w_bits, w_per_row=per_row, a_act=oracle.HRELU)
    assert np.array_equal(oi.cpu().numpy(), acc_ref)
    assert rel_close(of.cpu().numpy(), out_ref)


def test_linear_host(mpq, cuda):
    c = inputs.config1()
    x = torch.from_numpy(c["x"]).pin_memory()
    w = torch.from_numpy(c["w"]).pin_memory()
    oi = torch.empty((64, 64), dtype=torch.int32).pin_memory()
    of = torch.empty((64, 64), dtype=torch.float32).pin_memory()
    mpq.linear_host(x, w, 2, 2, out_i32_host=oi, out_f32_host=of)
    acc_ref, out_ref, _, _ = oracle.linear(c["x"], c["w"], 2, 2)
    assert np.array_equal(oi.numpy(), acc_ref)
    assert rel_close(of.numpy(), out_ref)


def test_linear_host_row_blocks(mpq, cuda):
    """m >= 1024: the product runs in row blocks that are copied out while the next one computes
    (ragged last block, per-row weight ranges, both outputs, then the int32 output alone)."""
    m, n, k = 1100, 70, 200
    x = inputs.uniform_levels(6, 11, (m, k), 3)
    w = inputs.uniform_levels(6, 12, (n, k), 2)
    xh, wh = torch.from_numpy(x).pin_memory(), torch.from_numpy(w).pin_memory()
    acc_ref, out_ref, _, _ = oracle.linear(x, w, 3, 2, w_per_row=True, a_act=oracle.HRELU)
    oi = torch.full((m, n), -1, dtype=torch.int32).pin_memory()
    of = torch.full((m, n), float("nan"), dtype=torch.float32).pin_memory()
    mpq.linear_host(xh, wh, 3, 2, mpq.ACT_HRELU, mpq.SCALE_PER_ROW, out_i32_host=oi, out_f32_host=of)
    assert np.array_equal(oi.numpy(), acc_ref)
    assert rel_close(of.numpy(), out_ref)
    oi.fill_(-1)
    mpq.linear_host(xh, wh, 3, 2, mpq.ACT_HRELU, mpq.SCALE_PER_ROW, out_i32_host=oi)
    assert np.array_equal(oi.numpy(), acc_ref)


def test_add_relu(mpq, cuda):
    rng = np.random.default_rng(1)
    a = rng.standard_normal(10007).astype(np.float32)
    b = rng.standard_normal(10007).astype(np.float32)
    y = torch.empty(10007, dtype=torch.float32, device=cuda)
    mpq.add_relu(_dev(a, cuda), _dev(b, cuda), y)
    assert np.array_equal(y.cpu().numpy(), np.maximum(a + b, 0))
    mpq.add_relu(_dev(a, cuda), None, y)
    assert np.array_equal(y.cpu().numpy(), np.maximum(a, 0))


def test_popc_peak_probe(mpq, cuda):
    rate, mhz, sms = mpq.measure_popc_peak()
    assert sms >= 100 and 500 < mhz < 3000
    per_clk_sm = rate / (mhz * 1e6 * sms)
    assert 8 <= per_clk_sm <= 130          # lanes per clock per SM: a plausible pipe width


def test_pipe_probes_are_sane(mpq, cuda):
    """The roofline probes return rates in the range the SM's unit counts allow: the instruction mix
    can only be slower than the plain population count, and the one-bit tensor instruction reports
    a positive, finite rate."""
    popc, mhz, sms = mpq.measure_popc_peak()
    assert sms > 0 and 500 < mhz < 3000
    lanes = popc / (mhz * 1e6 * sms)
    assert 8 < lanes < 40                                    # POPC results per clock per SM
    prev = None
    for L in (0, 4, 8):
        rate, _, _ = mpq.measure_mix_peak(L)
        assert 0 < rate <= popc * 1.05
        assert prev is None or rate <= prev * 1.05           # more logic per group never issues faster
        prev = rate
    for and_popc in (False, True):
        rate, mhz_b, _ = mpq.measure_b1_mma_peak(and_popc)
        per_clk = rate / (mhz_b * 1e6 * sms)
        assert 0 < per_clk < 8                               # warp instructions per clock per SM
