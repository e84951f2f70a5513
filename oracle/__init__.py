"""CPU oracle for the {-1,+1} encoded quantized layer -- TEST INFRASTRUCTURE ONLY.

Thin numpy front-end over ``mpq_oracle.c`` (plain C, built with gcc).  The
product path never imports this package: only the tests, the smoke check and
the benchmark's CPU-baseline leg do.  Nothing here is shared with the CUDA
sources; the two sides meet only in the tests, on the same seeded inputs.

Functions follow the paper's order: range (max-abs, or HReLU's positive side,
Table 1) -> quantizer (Eq. 15, Table 2, Eq. 20) -> integer layer product
(Eq. 1-2) -> decoder scale (Eq. 18).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mpq_oracle.c")
_LIB = os.path.join(_HERE, "libmpq_oracle.so")
_lock = threading.Lock()
_lib = None

HTANH, HRELU = 0, 1


def build(force: bool = False) -> str:
    """Compile the C oracle.  Strict IEEE: no fast-math, no FMA contraction."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fno-fast-math", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            i64, i32, f32 = ctypes.c_int64, ctypes.c_int, ctypes.c_float
            P = ctypes.c_void_p
            lib.mpq_oracle_absmax.argtypes = [P, i64, i64, i64, i32, i32, P]
            lib.mpq_oracle_absmax.restype = None
            lib.mpq_oracle_quantize.argtypes = [P, i64, i64, i64, P, i32, i32, i32, P]
            lib.mpq_oracle_quantize.restype = None
            lib.mpq_oracle_quantize_trig.argtypes = [P, i64, i64, i64, P, i32, i32, i32, P]
            lib.mpq_oracle_quantize_trig.restype = None
            lib.mpq_oracle_gemm.argtypes = [P, P, i64, i64, i64, P]
            lib.mpq_oracle_gemm.restype = i64
            lib.mpq_oracle_conv.argtypes = [P, i64, i64, i64, i64, P, i64, i64, i64, i64, i64, P]
            lib.mpq_oracle_conv.restype = i64
            lib.mpq_oracle_deconv.argtypes = [P, i64, i64, i64, i64, P, i64, i64, i64, i64, i64, P]
            lib.mpq_oracle_deconv.restype = i64
            lib.mpq_oracle_conv_at.argtypes = [P, i64, i64, i64, P, i64, i64, i64, i64, i64, i64, i64, i64]
            lib.mpq_oracle_conv_at.restype = i64
            lib.mpq_oracle_scale.argtypes = [P, i64, i64, i64, f32, P, i32, i32, i32, P]
            lib.mpq_oracle_scale.restype = None
            lib.mpq_oracle_scale_f64.argtypes = [P, i64, i64, i64, f32, P, i32, i32, i32, P]
            lib.mpq_oracle_scale_f64.restype = None
            lib.mpq_oracle_stem.argtypes = [P, P, i64, i64, i64, i32, P]
            lib.mpq_oracle_stem.restype = None
            lib.mpq_oracle_maxpool3x3s2.argtypes = [P, i64, i64, i64, P]
            lib.mpq_oracle_maxpool3x3s2.restype = None
            _lib = lib
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _f32c(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def threads() -> int:
    """Host threads the OpenMP loops will use (the cores this job may run on)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env)
    return len(os.sched_getaffinity(0))


def absmax(x, per_row: bool = False, act: int = HTANH) -> np.ndarray:
    """Range of a [rows x k] matrix: max|x| (or max of the positive side for HReLU)."""
    x = _f32c(x)
    x2 = x.reshape(x.shape[0], -1) if per_row else x.reshape(1, -1)
    out = np.zeros(x2.shape[0] if per_row else 1, dtype=np.float32)
    _load().mpq_oracle_absmax(_p(x2), x2.shape[0], x2.shape[1], x2.shape[1], int(per_row), int(act), _p(out))
    return out


def quantize(x, scale, bits: int, per_row: bool = False, act: int = HTANH) -> np.ndarray:
    """Float tensor -> odd integers q in [-(2^b-1), 2^b-1] (Eq. 15 / Table 2 / Eq. 20).

    ``x`` keeps its shape; with ``per_row`` the scale has one entry per slice of
    the leading axis, otherwise a single entry.
    """
    if not 1 <= bits <= 8:
        raise ValueError("bits must be in 1..8")
    x = _f32c(x)
    scale = _f32c(np.atleast_1d(scale))
    rows = x.shape[0] if per_row else 1
    k = x.size // rows if rows else 0
    if scale.size != rows:
        raise ValueError("scale has %d entries, expected %d" % (scale.size, rows))
    q = np.empty(x.shape, dtype=np.int16)
    _load().mpq_oracle_quantize(_p(x), rows, k, k, _p(scale), int(per_row), bits, int(act), _p(q))
    return q


def quantize_trig(x, scale, bits: int, per_row: bool = False, act: int = HTANH) -> np.ndarray:
    """The same codes through the trigonometric encoders (Eq. 11 and its family): each bit is the
    sign of a sine of x/s.  Equal to :func:`quantize` except within a rounding of a level boundary."""
    if not 1 <= bits <= 8:
        raise ValueError("bits must be in 1..8")
    x = _f32c(x)
    scale = _f32c(np.atleast_1d(scale))
    rows = x.shape[0] if per_row else 1
    k = x.size // rows if rows else 0
    if scale.size != rows:
        raise ValueError("scale has %d entries, expected %d" % (scale.size, rows))
    q = np.empty(x.shape, dtype=np.int16)
    _load().mpq_oracle_quantize_trig(_p(x), rows, k, k, _p(scale), int(per_row), bits, int(act), _p(q))
    return q


def levels(q: np.ndarray, bits: int) -> np.ndarray:
    """Odd integer q -> level index u = (q + 2^b - 1) / 2 whose bits are the code (Eq. 10)."""
    return (q.astype(np.int32) + ((1 << bits) - 1)) // 2


def gemm(qa, qb) -> np.ndarray:
    """acc[r][c] = sum_t qa[r][t] * qb[c][t] (Eq. 1-2), int32; raises if int32 overflows."""
    qa = np.ascontiguousarray(qa, dtype=np.int16)
    qb = np.ascontiguousarray(qb, dtype=np.int16)
    m, k = qa.shape
    n, k2 = qb.shape
    if k != k2:
        raise ValueError("inner sizes differ")
    acc = np.empty((m, n), dtype=np.int32)
    if _load().mpq_oracle_gemm(_p(qa), _p(qb), m, n, k, _p(acc)):
        raise OverflowError("accumulator does not fit int32")
    return acc


def conv(qx, qw, stride: int = 1, pad: int = 0) -> np.ndarray:
    """Direct convolution of decoded integers, NCHW x OIHW -> [N][O][Ho][Wo] int32."""
    qx = np.ascontiguousarray(qx, dtype=np.int16)
    qw = np.ascontiguousarray(qw, dtype=np.int16)
    N, C, H, W = qx.shape
    O, C2, KH, KW = qw.shape
    if C != C2:
        raise ValueError("channel counts differ")
    Ho = (H + 2 * pad - KH) // stride + 1
    Wo = (W + 2 * pad - KW) // stride + 1
    acc = np.empty((N, O, Ho, Wo), dtype=np.int32)
    if _load().mpq_oracle_conv(_p(qx), N, C, H, W, _p(qw), O, KH, KW, stride, pad, _p(acc)):
        raise OverflowError("accumulator does not fit int32")
    return acc


def deconv(qx, qw, stride: int = 2, pad: int = 0) -> np.ndarray:
    """Deconvolution (transposed convolution) of decoded integers: qx [N][C][H][W], qw [O][C][KH][KW]
    (output channel first) -> [N][O][Ho][Wo] int32 with Ho = (H - 1) stride - 2 pad + KH."""
    qx = np.ascontiguousarray(qx, dtype=np.int16)
    qw = np.ascontiguousarray(qw, dtype=np.int16)
    N, C, H, W = qx.shape
    O, C2, KH, KW = qw.shape
    if C != C2:
        raise ValueError("channel counts differ")
    Ho = (H - 1) * stride - 2 * pad + KH
    Wo = (W - 1) * stride - 2 * pad + KW
    if Ho <= 0 or Wo <= 0:
        raise ValueError("empty output")
    acc = np.empty((N, O, Ho, Wo), dtype=np.int32)
    if _load().mpq_oracle_deconv(_p(qx), N, C, H, W, _p(qw), O, KH, KW, stride, pad, _p(acc)):
        raise OverflowError("accumulator does not fit int32")
    return acc


def conv_at(qx, qw, stride: int, pad: int, b: int, o: int, oh: int, ow: int) -> int:
    """One output element of :func:`conv` (for sampling a large layer)."""
    qx = np.ascontiguousarray(qx, dtype=np.int16)
    qw = np.ascontiguousarray(qw, dtype=np.int16)
    _, C, H, W = qx.shape
    _, _, KH, KW = qw.shape
    return int(_load().mpq_oracle_conv_at(_p(qx), C, H, W, _p(qw), KH, KW, stride, pad, b, o, oh, ow))


def _scale_args(acc, s_w):
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    if acc.ndim == 2:
        outer, channels, inner = acc.shape[0], acc.shape[1], 1
    elif acc.ndim == 4:
        outer, channels, inner = acc.shape[0], acc.shape[1], acc.shape[2] * acc.shape[3]
    else:
        raise ValueError("acc must be [m][n] or [N][O][Ho][Wo]")
    s_w = _f32c(np.atleast_1d(s_w))
    per_channel = s_w.size != 1
    if per_channel and s_w.size != channels:
        raise ValueError("s_w has %d entries, expected 1 or %d" % (s_w.size, channels))
    return acc, outer, channels, inner, s_w, per_channel


def scale(acc, s_a: float, s_w, a_bits: int, w_bits: int) -> np.ndarray:
    """Decoder scale (Eq. 18) in fp32: float(acc) * ((s_a/L_a) * (s_w[c]/L_w))."""
    acc, outer, channels, inner, s_w, per_channel = _scale_args(acc, s_w)
    out = np.empty(acc.shape, dtype=np.float32)
    _load().mpq_oracle_scale(_p(acc), outer, channels, inner, float(np.float32(s_a)), _p(s_w),
                             int(per_channel), a_bits, w_bits, _p(out))
    return out


def scale_f64(acc, s_a: float, s_w, a_bits: int, w_bits: int) -> np.ndarray:
    """Decoder scale (Eq. 18) evaluated in double."""
    acc, outer, channels, inner, s_w, per_channel = _scale_args(acc, s_w)
    out = np.empty(acc.shape, dtype=np.float64)
    _load().mpq_oracle_scale_f64(_p(acc), outer, channels, inner, float(np.float32(s_a)), _p(s_w),
                                 int(per_channel), a_bits, w_bits, _p(out))
    return out


def epilogue(out, bias=None, residual=None, relu: bool = False) -> np.ndarray:
    """Glue after the decoder of a chained layer (not part of the paper's method, which has no bias):
    out + bias[c] (one rounded fp32 add), + residual (one rounded fp32 add), then max(., 0).
    ``out`` is [m][n] (bias per column) or [N][O][Ho][Wo] (bias per channel)."""
    f = np.array(out, dtype=np.float32, copy=True)
    if bias is not None:
        b = _f32c(bias)
        f = (f + (b[None, :] if f.ndim == 2 else b[None, :, None, None])).astype(np.float32)
    if residual is not None:
        f = (f + _f32c(residual)).astype(np.float32)
    if relu:
        f = np.where(f > 0, f, np.float32(0)).astype(np.float32)
    return f


def linear(x, w, a_bits: int, w_bits: int, w_per_row: bool = False, a_act: int = HTANH):
    """Whole encoded fully-connected layer (Fig. 1): returns (acc int32, out fp32, s_a, s_w)."""
    s_a = absmax(x, per_row=False, act=a_act)
    s_w = absmax(w, per_row=w_per_row)
    qa = quantize(x, s_a, a_bits, act=a_act)
    qb = quantize(w, s_w, w_bits, per_row=w_per_row)
    acc = gemm(qa, qb)
    return acc, scale(acc, s_a[0], s_w, a_bits, w_bits), s_a, s_w


def conv_layer(x, w, a_bits: int, w_bits: int, stride: int = 1, pad: int = 0,
               w_per_channel: bool = True, a_act: int = HTANH):
    """Whole encoded convolution layer: returns (acc int32, out fp32, s_a, s_w)."""
    s_a = absmax(x, per_row=False, act=a_act)
    s_w = absmax(w, per_row=w_per_channel)
    qx = quantize(x, s_a, a_bits, act=a_act)
    qw = quantize(w, s_w, w_bits, per_row=w_per_channel)
    acc = conv(qx, qw, stride, pad)
    return acc, scale(acc, s_a[0], s_w, a_bits, w_bits), s_a, s_w


def deconv_layer(x, w, a_bits: int, w_bits: int, stride: int = 2, pad: int = 0,
                 w_per_channel: bool = True, a_act: int = HTANH):
    """Whole encoded deconvolution layer, weights [O][C][KH][KW]: returns (acc int32, out fp32, s_a, s_w)."""
    s_a = absmax(x, per_row=False, act=a_act)
    s_w = absmax(w, per_row=w_per_channel)
    qx = quantize(x, s_a, a_bits, act=a_act)
    qw = quantize(w, s_w, w_bits, per_row=w_per_channel)
    acc = deconv(qx, qw, stride, pad)
    return acc, scale(acc, s_a[0], s_w, a_bits, w_bits), s_a, s_w


def stem(x, w, relu: bool = True) -> np.ndarray:
    """fp32 glue of the test network: 7x7 stride-2 pad-3 convolution, 3 -> 64 channels, each output one
    chain of fused multiply-adds over (c, kh, kw); then max(.,0)."""
    x, w = _f32c(x), _f32c(w)
    N, C, H, W = x.shape
    if C != 3 or w.shape != (64, 3, 7, 7):
        raise ValueError("stem takes [N][3][H][W] and a [64][3][7][7] weight")
    y = np.empty((N, 64, (H - 1) // 2 + 1, (W - 1) // 2 + 1), dtype=np.float32)
    _load().mpq_oracle_stem(_p(x), _p(w), N, H, W, int(relu), _p(y))
    return y


def maxpool3x3s2(x) -> np.ndarray:
    """3x3 max-pool, stride 2, pad 1 on [N][C][H][W]."""
    x = _f32c(x)
    N, C, H, W = x.shape
    y = np.empty((N, C, (H - 1) // 2 + 1, (W - 1) // 2 + 1), dtype=np.float32)
    _load().mpq_oracle_maxpool3x3s2(_p(x), N * C, H, W, _p(y))
    return y
