"""Binding of libmpq_context.so: the decoded-integer tensor-core comparison kernel (tcgen05 kind::i8).

Context for the benchmark tables only -- what the product of the decoded integers costs on the
5th-generation tensor cores, beside the bit-plane path.  Not part of the library's path and never
called by it."""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmpq_context.so")
_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libmpq_context.so is not built: run `python -m paper_1905_13389_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        i64, i32, P = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p
        L.mpqctx_i8_gemm.argtypes = [P, P, i64, i64, i64, P, i32, P, P, i32, i32, P, P]
        L.mpqctx_i8_gemm.restype = i32
        L.mpqctx_row_sums_u8.argtypes = [P, i64, i64, P, P]
        L.mpqctx_row_sums_u8.restype = i32
        _lib = L
    return _lib


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def row_sums_u8(u: torch.Tensor) -> torch.Tensor:
    rows, k = u.shape
    out = torch.empty(rows, dtype=torch.int32, device=u.device)
    rc = lib().mpqctx_row_sums_u8(u.data_ptr(), rows, k, out.data_ptr(), _stream())
    if rc:
        raise RuntimeError("mpqctx_row_sums_u8 failed with status %d" % rc)
    return out


def i8_gemm(a: torch.Tensor, b: torch.Tensor, out: torch.Tensor, error_flag: torch.Tensor,
            unsigned_levels=None, sums=None):
    """out[m][n] = sum_t a[m][t] * b[n][t] on int8 tensors (signed form), or -- with
    ``unsigned_levels = (L_a, L_b)`` and ``sums = (row sums of a, row sums of b)`` on uint8 level indices
    -- the product of the decoded levels q = 2u - L via Eq. 17's correction terms."""
    m, k = a.shape
    n = b.shape[0]
    if unsigned_levels is None:
        rc = lib().mpqctx_i8_gemm(a.data_ptr(), b.data_ptr(), m, n, k, out.data_ptr(), 0, None, None, 0, 0,
                                  error_flag.data_ptr(), _stream())
    else:
        rc = lib().mpqctx_i8_gemm(a.data_ptr(), b.data_ptr(), m, n, k, out.data_ptr(), 1, sums[0].data_ptr(),
                                  sums[1].data_ptr(), unsigned_levels[0], unsigned_levels[1],
                                  error_flag.data_ptr(), _stream())
    if rc:
        raise RuntimeError("mpqctx_i8_gemm failed with status %d" % rc)
    return out
