"""Thin Python binding of libmpq.so: argument marshalling only.

Every function has the name and the argument order of its C entry point in
``include/mpq.h`` (minus the ``mpq_`` prefix) and takes torch CUDA tensors where
the C side takes device pointers.  torch is used for device memory and streams
only; every step of the path runs in the library's own kernels.  There is no CPU
fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmpq.so")

OK = 0
SCALE_PER_TENSOR, SCALE_PER_ROW = 0, 1
ACT_HTANH, ACT_HRELU = 0, 1
ENC_LEVELS, ENC_TRIG = 0, 1

_lib = None


class MpqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s (status %d)" % (where, status_string(status), status))


def lib() -> ctypes.CDLL:
    """Loads libmpq.so (must have been built in-tree, see ``build.py``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libmpq.so is not built: run `python -m paper_1905_13389_b200.build` "
                              "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        i64, i32, P = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p
        L.mpq_status_string.argtypes = [i32]
        L.mpq_status_string.restype = ctypes.c_char_p
        L.mpq_row_words.argtypes = [i64]
        L.mpq_row_words.restype = i64
        L.mpq_packed_words.argtypes = [i64, i64, i32]
        L.mpq_packed_words.restype = i64
        L.mpq_absmax.argtypes = [P, i64, i64, i64, i32, i32, P, P]
        L.mpq_encode.argtypes = [P, i64, i64, i64, P, i32, i32, i32, P, P]
        L.mpq_encode_with.argtypes = [i32, P, i64, i64, i64, P, i32, i32, i32, P, P]
        L.mpq_encode_ranged.argtypes = [P, i64, i64, i64, i32, i32, P, P, P]
        L.mpq_encode_nchw.argtypes = [P, i32, i32, i32, i32, P, i32, i32, P, P]
        L.mpq_encode_oihw.argtypes = [P, i32, i32, i32, i32, P, i32, i32, P, P, P]
        L.mpq_gemm.argtypes = [P, i32, P, i32, i64, i64, i64, P, P, i64, P, P, i32, P]
        L.mpq_gemm_fused.argtypes = [P, i32, P, i32, i64, i64, i64, P, P, i64, P, P, i32, P, P, i32, P]
        L.mpq_conv.argtypes = [P, i32, i32, i32, i32, i32, P, i32, P, i32, i32, i32, i32, i32, P, P, P, P, i32, P]
        L.mpq_conv_encoded.argtypes = [P, i32, i32, i32, i32, i32, P, i32, P, i32, i32, i32, i32, i32, P, P, P, P, i32,
                                       P, i32, P, P, i32, i32, P, P]
        L.mpq_add_relu.argtypes = [P, P, P, i64, P]
        L.mpq_stem_conv7x7.argtypes = [P, P, P, i32, i32, i32, i32, P]
        L.mpq_maxpool3x3s2.argtypes = [P, P, i32, i32, i32, i32, P, P]
        L.mpq_conv_fused.argtypes = [P, i32, i32, i32, i32, i32, P, i32, P, i32, i32, i32, i32, i32, P, P, P, P, i32,
                                     P, i32, P, P]
        L.mpq_deconv.argtypes = [P, i32, i32, i32, i32, i32, P, i32, P, i32, i32, i32, i32, i32, P, P, P, P, i32,
                                 P, i32, P, P]
        L.mpq_deconv_weight_words.argtypes = [i32, i32, i32, i32, i32, i32]
        L.mpq_deconv_weight_words.restype = i64
        L.mpq_encode_deconv_weights.argtypes = [P, i32, i32, i32, i32, i32, P, i32, i32, P, P, P]
        L.mpq_zero.argtypes = [P, i64, P]
        L.mpq_linear_workspace.argtypes = [i64, i64, i64, i32, i32]
        L.mpq_linear_workspace.restype = i64
        L.mpq_linear.argtypes = [P, P, i64, i64, i64, i32, i32, i32, i32, P, P, P, i64, P]
        L.mpq_linear_static.argtypes = [P, P, i64, i64, i64, i32, i32, i32, i32, P, P, P]
        L.mpq_linear_host_workspace.argtypes = [i64, i64, i64, i32, i32]
        L.mpq_linear_host_workspace.restype = i64
        L.mpq_linear_host.argtypes = [P, P, i64, i64, i64, i32, i32, i32, i32, P, P, P, i64, P]
        L.mpq_linear_host_prepared_workspace.argtypes = [i64, i64, i64, i32]
        L.mpq_linear_host_prepared_workspace.restype = i64
        L.mpq_linear_host_prepared.argtypes = [P, P, P, i64, i64, i64, i32, i32, i32, i32, P, P, P, i64, P]
        L.mpq_measure_popc_peak.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double),
                                            ctypes.POINTER(ctypes.c_int), P]
        L.mpq_measure_mix_peak.argtypes = [i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double),
                                           ctypes.POINTER(ctypes.c_int), P]
        L.mpq_measure_mix_peak.restype = i32
        L.mpq_measure_b1_mma_peak.argtypes = [i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double),
                                              ctypes.POINTER(ctypes.c_int), P]
        L.mpq_measure_b1_mma_peak.restype = i32
        for name in ("mpq_absmax", "mpq_encode", "mpq_encode_nchw", "mpq_encode_oihw", "mpq_gemm", "mpq_conv",
                     "mpq_add_relu", "mpq_stem_conv7x7", "mpq_maxpool3x3s2", "mpq_conv_fused", "mpq_zero", "mpq_linear", "mpq_linear_static", "mpq_linear_host", "mpq_measure_popc_peak",
                     "mpq_encode_with", "mpq_encode_ranged", "mpq_gemm_fused", "mpq_conv_encoded", "mpq_linear_host_prepared",
                     "mpq_deconv", "mpq_encode_deconv_weights"):
            getattr(L, name).restype = i32
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().mpq_status_string(int(status)).decode()


def row_words(k: int) -> int:
    return int(lib().mpq_row_words(k))


def packed_words(rows: int, k: int, bits: int) -> int:
    return int(lib().mpq_packed_words(rows, k, bits))


def _check(status: int, where: str):
    if status != OK:
        raise MpqError(status, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor], dtype=None) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError("expected dtype %s, got %s" % (dtype, t.dtype))
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    return t.data_ptr()


def absmax(x: torch.Tensor, mode: int = SCALE_PER_TENSOR, act: int = ACT_HTANH,
           out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Range of a float tensor viewed as [rows x k] (rows = leading axis): 1 or rows values."""
    rows = x.shape[0]
    k = x.numel() // rows
    if out is None:
        out = torch.empty(rows if mode == SCALE_PER_ROW else 1, dtype=torch.float32, device=x.device)
    _check(lib().mpq_absmax(_ptr(x, torch.float32), rows, k, k, mode, act, _ptr(out, torch.float32), _stream()),
           "mpq_absmax")
    return out


def encode(x: torch.Tensor, scale: torch.Tensor, bits: int, mode: int = SCALE_PER_TENSOR,
           act: int = ACT_HTANH, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """[rows x k] fp32 -> planes [bits][rows][row_words(k)] (int32 storage of the uint32 words)."""
    rows, k = x.shape
    if out is None:
        out = torch.empty((bits, rows, row_words(k)), dtype=torch.int32, device=x.device)
    _check(lib().mpq_encode(_ptr(x, torch.float32), rows, k, k, _ptr(scale, torch.float32), mode, act, bits,
                            _ptr(out, torch.int32), _stream()), "mpq_encode")
    return out


def encode_ranged(x: torch.Tensor, bits: int, act: int = ACT_HTANH):
    """Per-row ranges and planes of [rows x k] in one pass over memory: returns (scale [rows], planes)."""
    rows, k = x.shape
    scale = torch.empty(rows, dtype=torch.float32, device=x.device)
    planes = torch.empty((bits, rows, row_words(k)), dtype=torch.int32, device=x.device)
    _check(lib().mpq_encode_ranged(_ptr(x, torch.float32), rows, k, k, act, bits, _ptr(scale, torch.float32),
                                   _ptr(planes, torch.int32), _stream()), "mpq_encode_ranged")
    return scale, planes


def encode_with(encoder: int, x: torch.Tensor, scale: torch.Tensor, bits: int, mode: int = SCALE_PER_TENSOR,
                act: int = ACT_HTANH, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """:func:`encode` with the form of the Encoder selectable: ENC_LEVELS or ENC_TRIG (Eq. 11's sines)."""
    rows, k = x.shape
    if out is None:
        out = torch.empty((bits, rows, row_words(k)), dtype=torch.int32, device=x.device)
    _check(lib().mpq_encode_with(encoder, _ptr(x, torch.float32), rows, k, k, _ptr(scale, torch.float32), mode, act,
                                 bits, _ptr(out, torch.int32), _stream()), "mpq_encode_with")
    return out


def encode_nchw(x: torch.Tensor, scale: torch.Tensor, bits: int, act: int = ACT_HTANH,
                out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """[N][C][H][W] fp32 -> planes [bits][N][H][W][C/32]."""
    N, C, H, W = x.shape
    if out is None:
        out = torch.empty((bits, N, H, W, max(C // 32, 1)), dtype=torch.int32, device=x.device)
    _check(lib().mpq_encode_nchw(_ptr(x, torch.float32), N, C, H, W, _ptr(scale, torch.float32), act, bits,
                                 _ptr(out, torch.int32), _stream()), "mpq_encode_nchw")
    return out


def encode_oihw(w: torch.Tensor, scale: torch.Tensor, bits: int, mode: int = SCALE_PER_ROW):
    """[O][C][KH][KW] fp32 -> (planes [bits][O][row_words(KH*KW*C)], tap_sums [KH*KW][O])."""
    O, C, KH, KW = w.shape
    planes = torch.empty((bits, O, row_words(KH * KW * C)), dtype=torch.int32, device=w.device)
    tap_sums = torch.empty((KH * KW, O), dtype=torch.int32, device=w.device)
    _check(lib().mpq_encode_oihw(_ptr(w, torch.float32), O, C, KH, KW, _ptr(scale, torch.float32), mode, bits,
                                 _ptr(planes, torch.int32), _ptr(tap_sums, torch.int32), _stream()),
           "mpq_encode_oihw")
    return planes, tap_sums


def gemm(a_planes: torch.Tensor, a_bits: int, b_planes: torch.Tensor, b_bits: int, m: int, n: int, k: int,
         c_i32: Optional[torch.Tensor] = None, c_f32: Optional[torch.Tensor] = None,
         a_scale: Optional[torch.Tensor] = None, b_scale: Optional[torch.Tensor] = None,
         b_mode: int = SCALE_PER_TENSOR):
    """C = A B^T on packed planes; writes the int32 accumulators and/or the scaled fp32 output."""
    ldc = n
    _check(lib().mpq_gemm(_ptr(a_planes, torch.int32), a_bits, _ptr(b_planes, torch.int32), b_bits, m, n, k,
                          _ptr(c_i32, torch.int32), _ptr(c_f32, torch.float32), ldc,
                          _ptr(a_scale, torch.float32), _ptr(b_scale, torch.float32), b_mode, _stream()),
           "mpq_gemm")
    return c_i32, c_f32


def gemm_fused(a_planes: torch.Tensor, a_bits: int, b_planes: torch.Tensor, b_bits: int, m: int, n: int, k: int,
               c_i32: Optional[torch.Tensor] = None, c_f32: Optional[torch.Tensor] = None,
               a_scale: Optional[torch.Tensor] = None, b_scale: Optional[torch.Tensor] = None,
               b_mode: int = SCALE_PER_TENSOR, bias: Optional[torch.Tensor] = None,
               residual: Optional[torch.Tensor] = None, relu: bool = False):
    """:func:`gemm` with bias, residual and max(., 0) folded into the store."""
    _check(lib().mpq_gemm_fused(_ptr(a_planes, torch.int32), a_bits, _ptr(b_planes, torch.int32), b_bits, m, n, k,
                                _ptr(c_i32, torch.int32), _ptr(c_f32, torch.float32), n,
                                _ptr(a_scale, torch.float32), _ptr(b_scale, torch.float32), b_mode,
                                _ptr(bias, torch.float32), _ptr(residual, torch.float32), int(relu), _stream()),
           "mpq_gemm_fused")
    return c_i32, c_f32


def conv(x_planes: torch.Tensor, a_bits: int, N: int, C: int, H: int, W: int,
         w_planes: torch.Tensor, w_bits: int, tap_sums: Optional[torch.Tensor],
         O: int, KH: int, KW: int, stride: int, pad: int,
         y_i32: Optional[torch.Tensor] = None, y_f32: Optional[torch.Tensor] = None,
         x_scale: Optional[torch.Tensor] = None, w_scale: Optional[torch.Tensor] = None,
         w_mode: int = SCALE_PER_ROW):
    """Implicit-im2col convolution on packed planes; y is [N][O][Ho][Wo]."""
    _check(lib().mpq_conv(_ptr(x_planes, torch.int32), a_bits, N, C, H, W, _ptr(w_planes, torch.int32), w_bits,
                          _ptr(tap_sums, torch.int32), O, KH, KW, stride, pad,
                          _ptr(y_i32, torch.int32), _ptr(y_f32, torch.float32),
                          _ptr(x_scale, torch.float32), _ptr(w_scale, torch.float32), w_mode, _stream()),
           "mpq_conv")
    return y_i32, y_f32


def conv_fused(x_planes: torch.Tensor, a_bits: int, N: int, C: int, H: int, W: int,
               w_planes: torch.Tensor, w_bits: int, tap_sums: Optional[torch.Tensor],
               O: int, KH: int, KW: int, stride: int, pad: int,
               y_i32: Optional[torch.Tensor], y_f32: torch.Tensor,
               x_scale: torch.Tensor, w_scale: torch.Tensor, w_mode: int = SCALE_PER_ROW,
               residual: Optional[torch.Tensor] = None, relu: bool = False,
               out_max: Optional[torch.Tensor] = None):
    """:func:`conv` with residual add, max(., 0) and the next layer's range folded into the store."""
    _check(lib().mpq_conv_fused(_ptr(x_planes, torch.int32), a_bits, N, C, H, W, _ptr(w_planes, torch.int32), w_bits,
                                _ptr(tap_sums, torch.int32), O, KH, KW, stride, pad,
                                _ptr(y_i32, torch.int32), _ptr(y_f32, torch.float32),
                                _ptr(x_scale, torch.float32), _ptr(w_scale, torch.float32), w_mode,
                                _ptr(residual, torch.float32), int(relu), _ptr(out_max, torch.float32), _stream()),
           "mpq_conv_fused")
    return y_i32, y_f32


def conv_encoded(x_planes: torch.Tensor, a_bits: int, N: int, C: int, H: int, W: int,
                 w_planes: torch.Tensor, w_bits: int, tap_sums: Optional[torch.Tensor],
                 O: int, KH: int, KW: int, stride: int, pad: int,
                 y_i32: Optional[torch.Tensor], y_f32: Optional[torch.Tensor],
                 x_scale: torch.Tensor, w_scale: torch.Tensor, w_mode: int,
                 residual: Optional[torch.Tensor], relu: bool, out_max: Optional[torch.Tensor],
                 next_scale: torch.Tensor, next_act: int, next_bits: int,
                 next_planes: Optional[torch.Tensor] = None) -> torch.Tensor:
    """:func:`conv_fused` whose store also runs the consumer's Encoder with a range known beforehand:
    returns next_planes [next_bits][N][Ho][Wo][O/32]; y_f32 may be None."""
    Ho, Wo = (H + 2 * pad - KH) // stride + 1, (W + 2 * pad - KW) // stride + 1
    if next_planes is None:
        next_planes = torch.empty((next_bits, N, Ho, Wo, O // 32), dtype=torch.int32, device=x_planes.device)
    _check(lib().mpq_conv_encoded(_ptr(x_planes, torch.int32), a_bits, N, C, H, W, _ptr(w_planes, torch.int32), w_bits,
                                  _ptr(tap_sums, torch.int32), O, KH, KW, stride, pad,
                                  _ptr(y_i32, torch.int32), _ptr(y_f32, torch.float32),
                                  _ptr(x_scale, torch.float32), _ptr(w_scale, torch.float32), w_mode,
                                  _ptr(residual, torch.float32), int(relu), _ptr(out_max, torch.float32),
                                  _ptr(next_scale, torch.float32), next_act, next_bits,
                                  _ptr(next_planes, torch.int32), _stream()), "mpq_conv_encoded")
    return next_planes


def encode_deconv_weights(w: torch.Tensor, scale: torch.Tensor, bits: int, stride: int, mode: int = SCALE_PER_ROW):
    """Deconvolution filters [O][C][KH][KW] fp32 (output channel first) -> (planes, one packed matrix per
    filter phase, flat int32; tap_sums [KH*KW][O], taps counted phase by phase)."""
    O, C, KH, KW = w.shape
    words = lib().mpq_deconv_weight_words(O, C, KH, KW, stride, bits)
    if words <= 0:
        raise MpqError(3, "mpq_deconv_weight_words")          # MPQ_ERR_UNSUPPORTED: filter outside the supported set
    planes = torch.empty((words,), dtype=torch.int32, device=w.device)
    tap_sums = torch.empty((KH * KW, O), dtype=torch.int32, device=w.device)
    _check(lib().mpq_encode_deconv_weights(_ptr(w, torch.float32), O, C, KH, KW, stride, _ptr(scale, torch.float32),
                                           mode, bits, _ptr(planes, torch.int32), _ptr(tap_sums, torch.int32),
                                           _stream()), "mpq_encode_deconv_weights")
    return planes, tap_sums


def deconv(x_planes: torch.Tensor, a_bits: int, N: int, C: int, H: int, W: int,
           w_planes: torch.Tensor, w_bits: int, tap_sums: torch.Tensor,
           O: int, KH: int, KW: int, stride: int, pad: int,
           y_i32: Optional[torch.Tensor], y_f32: Optional[torch.Tensor],
           x_scale: Optional[torch.Tensor] = None, w_scale: Optional[torch.Tensor] = None,
           w_mode: int = SCALE_PER_ROW, residual: Optional[torch.Tensor] = None, relu: bool = False,
           out_max: Optional[torch.Tensor] = None):
    """Deconvolution (transposed convolution) on packed planes -> [N][O][Ho][Wo], Ho = (H-1)*stride - 2*pad + KH."""
    _check(lib().mpq_deconv(_ptr(x_planes, torch.int32), a_bits, N, C, H, W, _ptr(w_planes, torch.int32), w_bits,
                            _ptr(tap_sums, torch.int32), O, KH, KW, stride, pad,
                            _ptr(y_i32, torch.int32), _ptr(y_f32, torch.float32),
                            _ptr(x_scale, torch.float32), _ptr(w_scale, torch.float32), w_mode,
                            _ptr(residual, torch.float32), int(relu), _ptr(out_max, torch.float32), _stream()),
           "mpq_deconv")
    return y_i32, y_f32


def zero(t: torch.Tensor) -> torch.Tensor:
    """Zeroes a device tensor on the current stream (cudaMemsetAsync)."""
    _check(lib().mpq_zero(t.data_ptr(), t.numel() * t.element_size(), _stream()), "mpq_zero")
    return t


def add_relu(a: torch.Tensor, b: Optional[torch.Tensor], y: torch.Tensor) -> torch.Tensor:
    _check(lib().mpq_add_relu(_ptr(a, torch.float32), _ptr(b, torch.float32), _ptr(y, torch.float32),
                              a.numel(), _stream()), "mpq_add_relu")
    return y


def stem_conv7x7(x: torch.Tensor, w: torch.Tensor, relu: bool = True,
                 out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """fp32 stem: x [N][3][H][W], w [64][3][7][7] -> [N][64][Ho][Wo] (7x7, stride 2, pad 3)."""
    N, C, H, W = x.shape
    if C != 3 or tuple(w.shape) != (64, 3, 7, 7):
        raise ValueError("the stem takes 3 input channels and a [64][3][7][7] weight")
    if out is None:
        out = torch.empty((N, 64, (H - 1) // 2 + 1, (W - 1) // 2 + 1), dtype=torch.float32, device=x.device)
    _check(lib().mpq_stem_conv7x7(_ptr(x, torch.float32), _ptr(w, torch.float32), _ptr(out, torch.float32),
                                  N, H, W, int(relu), _stream()), "mpq_stem_conv7x7")
    return out


def maxpool3x3s2(x: torch.Tensor, out: Optional[torch.Tensor] = None,
                 out_max: Optional[torch.Tensor] = None) -> torch.Tensor:
    """3x3 max-pool, stride 2, pad 1 on [N][C][H][W]; out_max (zeroed 1-float tensor) is raised to max(y, 0)."""
    N, C, H, W = x.shape
    if out is None:
        out = torch.empty((N, C, (H - 1) // 2 + 1, (W - 1) // 2 + 1), dtype=torch.float32, device=x.device)
    _check(lib().mpq_maxpool3x3s2(_ptr(x, torch.float32), _ptr(out, torch.float32), N, C, H, W,
                                  _ptr(out_max, torch.float32), _stream()),
           "mpq_maxpool3x3s2")
    return out


def linear_workspace(m: int, n: int, k: int, a_bits: int, w_bits: int) -> int:
    return int(lib().mpq_linear_workspace(m, n, k, a_bits, w_bits))


def linear(x: torch.Tensor, w: torch.Tensor, a_bits: int, w_bits: int,
           a_act: int = ACT_HTANH, w_mode: int = SCALE_PER_TENSOR,
           out_i32: Optional[torch.Tensor] = None, out_f32: Optional[torch.Tensor] = None,
           workspace: Optional[torch.Tensor] = None):
    """Whole encoded fully-connected layer on device tensors: x [m x k], w [n x k] -> [m x n]."""
    m, k = x.shape
    n, _ = w.shape
    if workspace is None:
        workspace = torch.empty(linear_workspace(m, n, k, a_bits, w_bits), dtype=torch.uint8, device=x.device)
    _check(lib().mpq_linear(_ptr(x, torch.float32), _ptr(w, torch.float32), m, n, k, a_bits, w_bits, a_act, w_mode,
                            _ptr(out_i32, torch.int32), _ptr(out_f32, torch.float32),
                            workspace.data_ptr(), workspace.numel(), _stream()), "mpq_linear")
    return out_i32, out_f32


LINEAR_STATIC_BYTES = 16 * 1024 * 1024


def linear_static(x: torch.Tensor, w: torch.Tensor, a_bits: int, w_bits: int,
                  a_act: int = ACT_HTANH, w_mode: int = SCALE_PER_TENSOR,
                  out_i32: Optional[torch.Tensor] = None, out_f32: Optional[torch.Tensor] = None):
    """:func:`linear` for callers that may not allocate: the ranges and packed operands go to a
    buffer built into the library (LINEAR_STATIC_BYTES per GPU) instead of a workspace tensor.
    Calls on one device share that buffer, so do not let two of them overlap on the GPU."""
    m, k = x.shape
    n, _ = w.shape
    _check(lib().mpq_linear_static(_ptr(x, torch.float32), _ptr(w, torch.float32), m, n, k, a_bits, w_bits,
                                   a_act, w_mode, _ptr(out_i32, torch.int32), _ptr(out_f32, torch.float32),
                                   _stream()), "mpq_linear_static")
    return out_i32, out_f32


def linear_host_workspace(m: int, n: int, k: int, a_bits: int, w_bits: int) -> int:
    return int(lib().mpq_linear_host_workspace(m, n, k, a_bits, w_bits))


def linear_host(x_host: torch.Tensor, w_host: torch.Tensor, a_bits: int, w_bits: int,
                a_act: int = ACT_HTANH, w_mode: int = SCALE_PER_TENSOR,
                out_i32_host: Optional[torch.Tensor] = None, out_f32_host: Optional[torch.Tensor] = None,
                workspace: Optional[torch.Tensor] = None):
    """Whole encoded fully-connected layer from (pinned) host tensors; synchronizes the stream."""
    m, k = x_host.shape
    n, _ = w_host.shape
    need = linear_host_workspace(m, n, k, a_bits, w_bits)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device="cuda")
    for t in (x_host, w_host, out_i32_host, out_f32_host):
        if t is not None and (t.is_cuda or not t.is_contiguous()):
            raise ValueError("host tensors must be contiguous CPU tensors")
    hp = lambda t: None if t is None else t.data_ptr()
    _check(lib().mpq_linear_host(hp(x_host), hp(w_host), m, n, k, a_bits, w_bits, a_act, w_mode,
                                 hp(out_i32_host), hp(out_f32_host), workspace.data_ptr(), workspace.numel(),
                                 _stream()), "mpq_linear_host")
    return out_i32_host, out_f32_host


def linear_host_prepared_workspace(m: int, n: int, k: int, a_bits: int) -> int:
    return int(lib().mpq_linear_host_prepared_workspace(m, n, k, a_bits))


def linear_host_prepared(x_host: torch.Tensor, w_planes: torch.Tensor, w_scale: torch.Tensor, n: int,
                         a_bits: int, w_bits: int, a_act: int = ACT_HTANH, w_mode: int = SCALE_PER_TENSOR,
                         out_i32_host: Optional[torch.Tensor] = None, out_f32_host: Optional[torch.Tensor] = None,
                         workspace: Optional[torch.Tensor] = None):
    """:func:`linear_host` with the weights already packed on the device (encoded once): only the
    activations go up and the results come down; synchronizes the stream."""
    m, k = x_host.shape
    if workspace is None:
        workspace = torch.empty(linear_host_prepared_workspace(m, n, k, a_bits), dtype=torch.uint8, device=w_planes.device)
    for t in (x_host, out_i32_host, out_f32_host):
        if t is not None and (t.is_cuda or not t.is_contiguous()):
            raise ValueError("host tensors must be contiguous CPU tensors")
    hp = lambda t: None if t is None else t.data_ptr()
    _check(lib().mpq_linear_host_prepared(hp(x_host), _ptr(w_planes, torch.int32), _ptr(w_scale, torch.float32),
                                          m, n, k, a_bits, w_bits, a_act, w_mode, hp(out_i32_host), hp(out_f32_host),
                                          workspace.data_ptr(), workspace.numel(), _stream()), "mpq_linear_host_prepared")
    return out_i32_host, out_f32_host


def measure_popc_peak():
    """(lane-level POPC results per second over the chip, SM MHz seen by the probe, SM count)."""
    rate, mhz, sms = ctypes.c_double(), ctypes.c_double(), ctypes.c_int()
    _check(lib().mpq_measure_popc_peak(ctypes.byref(rate), ctypes.byref(mhz), ctypes.byref(sms), _stream()),
           "mpq_measure_popc_peak")
    return rate.value, mhz.value, sms.value


def measure_mix_peak(logic_per_popc: int = 4):
    """(groups per second of `logic_per_popc` logic ops + 1 POPC + 1 multiply-add, SM MHz, SM count)."""
    rate, mhz, sms = ctypes.c_double(), ctypes.c_double(), ctypes.c_int()
    _check(lib().mpq_measure_mix_peak(logic_per_popc, ctypes.byref(rate), ctypes.byref(mhz), ctypes.byref(sms),
                                      _stream()), "mpq_measure_mix_peak")
    return rate.value, mhz.value, sms.value


def measure_b1_mma_peak(and_popc: bool = False):
    """(warp-level mma.sync.m16n8k256 b1 instructions per second over the chip, SM MHz, SM count)."""
    rate, mhz, sms = ctypes.c_double(), ctypes.c_double(), ctypes.c_int()
    _check(lib().mpq_measure_b1_mma_peak(int(and_popc), ctypes.byref(rate), ctypes.byref(mhz), ctypes.byref(sms),
                                         _stream()), "mpq_measure_b1_mma_peak")
    return rate.value, mhz.value, sms.value
