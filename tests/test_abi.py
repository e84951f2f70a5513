"""The C-ABI boundary on a machine without a GPU: the library loads, exports every symbol the
header declares, answers its size queries, and rejects bad arguments before launching anything."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "mpq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mpq_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(mpq):
    names = _declared_functions()
    assert {"mpq_encode", "mpq_gemm", "mpq_conv", "mpq_absmax"} <= set(names)
    L = mpq.lib()
    for name in names:
        assert hasattr(L, name), name


def test_row_words_and_packed_words(mpq):
    """Bit-vector storage: bits/32 of the fp32 size plus row padding to 16 bytes."""
    assert [mpq.row_words(k) for k in (1, 32, 33, 128, 129, 4096, 9216)] == [4, 4, 4, 4, 8, 128, 288]
    assert mpq.row_words(0) == 0 and mpq.row_words(-5) == 0
    assert mpq.packed_words(4096, 9216, 2) == 2 * 4096 * 288
    for bits in range(1, 9):
        words = mpq.packed_words(1000, 4096, bits)
        assert words * 4 * 32 == bits * 1000 * 4096 * 4          # exactly 32/bits smaller than fp32
    assert mpq.packed_words(10, 10, 0) == 0 and mpq.packed_words(10, 10, 9) == 0
    assert mpq.packed_words(0, 10, 2) == 0


def test_status_strings(mpq):
    seen = {mpq.status_string(s) for s in range(8)}
    assert len(seen) == 8 and "ok" in seen
    assert mpq.status_string(99) == "unknown status"


def test_host_side_argument_checks(mpq):
    """Errors the host can see come back as a status before any launch (nothing here touches a GPU)."""
    L = mpq.lib()
    buf = (ctypes.c_uint32 * 64)()
    p = ctypes.cast(buf, ctypes.c_void_p)
    aligned = ctypes.c_void_p((p.value + 15) // 16 * 16)
    odd = ctypes.c_void_p(aligned.value + 4)
    NULL, ERR_NULL, ERR_SHAPE, ERR_UNSUP, ERR_OVER, ERR_ALIGN = None, 1, 2, 3, 4, 5
    # mpq_gemm
    assert L.mpq_gemm(NULL, 2, aligned, 2, 4, 4, 32, aligned, NULL, 4, NULL, NULL, 0, NULL) == ERR_NULL
    assert L.mpq_gemm(aligned, 2, aligned, 2, 4, 4, 32, NULL, NULL, 4, NULL, NULL, 0, NULL) == ERR_NULL
    assert L.mpq_gemm(aligned, 2, aligned, 2, 4, 4, 32, NULL, aligned, 4, NULL, NULL, 0, NULL) == ERR_NULL   # fp32 out needs scales
    assert L.mpq_gemm(aligned, 2, aligned, 2, 0, 4, 32, aligned, NULL, 4, NULL, NULL, 0, NULL) == ERR_SHAPE
    assert L.mpq_gemm(aligned, 2, aligned, 2, 4, 4, 32, aligned, NULL, 3, NULL, NULL, 0, NULL) == ERR_SHAPE   # ldc < n
    for bad in (0, 9, -1):
        assert L.mpq_gemm(aligned, bad, aligned, 2, 4, 4, 32, aligned, NULL, 4, NULL, NULL, 0, NULL) == ERR_UNSUP
        assert L.mpq_gemm(aligned, 2, aligned, bad, 4, 4, 32, aligned, NULL, 4, NULL, NULL, 0, NULL) == ERR_UNSUP
    assert L.mpq_gemm(aligned, 8, aligned, 8, 4, 4, 33026, aligned, NULL, 4, NULL, NULL, 0, NULL) == ERR_OVER
    assert L.mpq_gemm(aligned, 1, aligned, 1, 4, 4, 2 ** 31, aligned, NULL, 4, NULL, NULL, 0, NULL) == ERR_OVER
    assert L.mpq_gemm(odd, 2, aligned, 2, 4, 4, 32, aligned, NULL, 4, NULL, NULL, 0, NULL) == ERR_ALIGN
    # mpq_encode / mpq_absmax
    assert L.mpq_encode(NULL, 4, 32, 32, aligned, 0, 0, 2, aligned, NULL) == ERR_NULL
    assert L.mpq_encode(aligned, 4, 32, 16, aligned, 0, 0, 2, aligned, NULL) == ERR_SHAPE                    # ldx < k
    assert L.mpq_encode(aligned, 4, 32, 32, aligned, 0, 0, 9, aligned, NULL) == ERR_UNSUP
    assert L.mpq_encode(aligned, 4, 32, 32, aligned, 2, 0, 2, aligned, NULL) == ERR_UNSUP                    # bad scale mode
    assert L.mpq_encode(aligned, 4, 32, 32, aligned, 0, 7, 2, aligned, NULL) == ERR_UNSUP                    # bad activation
    assert L.mpq_encode(aligned, 4, 32, 32, aligned, 0, 0, 2, odd, NULL) == ERR_ALIGN
    assert L.mpq_absmax(NULL, 4, 32, 32, 0, 0, aligned, NULL) == ERR_NULL
    assert L.mpq_absmax(aligned, 4, 0, 32, 0, 0, aligned, NULL) == ERR_SHAPE
    # mpq_conv: 64 encoding choices, 1x1 / 3x3 kernels, stride 1 / 2, pad 0 / 1, C of 32, 64 or 128 j
    def conv(a_bits=2, C=64, w_bits=2, KH=3, KW=3, stride=1, pad=1, taps=aligned, x=aligned):
        return L.mpq_conv(x, a_bits, 1, C, 8, 8, aligned, w_bits, taps, 16, KH, KW, stride, pad,
                          aligned, NULL, NULL, NULL, 0, NULL)
    assert conv(x=NULL) == ERR_NULL
    assert conv(taps=NULL) == ERR_NULL                     # padding needs the tap sums
    assert conv(a_bits=0) == ERR_UNSUP and conv(w_bits=9) == ERR_UNSUP
    assert conv(KH=5, KW=5) == ERR_UNSUP and conv(KH=3, KW=1) == ERR_UNSUP
    assert conv(stride=3) == ERR_UNSUP and conv(pad=2) == ERR_UNSUP
    assert conv(C=48) == ERR_UNSUP and conv(C=96) == ERR_UNSUP
    assert conv(a_bits=8, w_bits=8, C=4096) == ERR_OVER    # 9 * 4096 * 255 * 255 >= 2^31
    assert L.mpq_encode_nchw(aligned, 1, 48, 4, 4, aligned, 0, 2, aligned, NULL) == ERR_UNSUP
    assert L.mpq_encode_oihw(aligned, 4, 64, 3, 3, aligned, 0, 2, aligned, NULL, NULL) == ERR_NULL
    # fused-store convolution: the glue needs the fp32 output
    assert L.mpq_conv_fused(aligned, 2, 1, 64, 8, 8, aligned, 2, aligned, 16, 3, 3, 1, 1, aligned, NULL,
                            NULL, NULL, 0, aligned, 1, NULL, NULL) == ERR_NULL
    assert L.mpq_zero(NULL, 4, NULL) == ERR_NULL and L.mpq_zero(aligned, 0, NULL) == ERR_SHAPE
    assert L.mpq_stem_conv7x7(NULL, aligned, aligned, 1, 8, 8, 1, NULL) == ERR_NULL
    assert L.mpq_maxpool3x3s2(aligned, aligned, 0, 4, 8, 8, NULL, NULL) == ERR_SHAPE
    assert L.mpq_measure_mix_peak(9, None, None, None, NULL) == ERR_UNSUP
    # whole-layer calls
    assert mpq.linear_workspace(4, 0, 4, 2, 2) == 0
    lw = mpq.linear_workspace(64, 64, 512, 2, 2)
    assert lw >= 2 * 2 * 64 * 16 * 4
    assert L.mpq_linear(aligned, aligned, 64, 64, 512, 2, 2, 0, 0, aligned, NULL, ctypes.c_void_p(256), lw - 1, NULL) == 7
    assert L.mpq_linear(aligned, aligned, 64, 64, 512, 2, 2, 0, 0, aligned, NULL, ctypes.c_void_p(260), lw, NULL) == ERR_ALIGN
    assert L.mpq_linear(aligned, aligned, 64, 64, 512, 2, 9, 0, 0, aligned, NULL, ctypes.c_void_p(256), lw, NULL) == ERR_UNSUP
    assert mpq.linear_host_workspace(0, 4, 4, 2, 2) == 0
    need = mpq.linear_host_workspace(64, 64, 512, 2, 2)
    assert need >= 2 * 64 * 512 * 4 + 2 * 64 * 64 * 4
    assert L.mpq_linear_host(aligned, aligned, 64, 64, 512, 2, 2, 0, 0, aligned, NULL, ctypes.c_void_p(256), need - 1, NULL) == 7
    assert L.mpq_linear_host(aligned, aligned, 64, 64, 512, 2, 2, 0, 0, NULL, NULL, ctypes.c_void_p(256), need, NULL) == ERR_NULL


def test_binding_refuses_cpu_tensors(mpq):
    """No CPU fallback: device entry points reject host tensors instead of computing elsewhere."""
    import torch
    x = torch.zeros((4, 32))
    with pytest.raises(ValueError):
        mpq._ptr(x, torch.float32)
