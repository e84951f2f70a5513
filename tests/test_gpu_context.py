"""The decoded-integer tensor-core comparison kernel (context for the benchmark, not the library's
path): its int32 product of the decoded levels must equal the oracle's integer GEMM, in the signed
form (codes of up to 7 bits held as int8) and in the unsigned form (8-bit level indices with the
correction terms of Eq. 17), and the bit-plane path must agree with it."""
import numpy as np
import pytest
import torch

import oracle
from paper_1905_13389_b200 import context, inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("m,n,k", [(128, 256, 128), (256, 768, 1024), (512, 256, 4096), (4096, 4096, 128)])
@pytest.mark.parametrize("a_bits,w_bits", [(2, 2), (4, 7), (7, 3)])
def test_signed_form_equals_the_oracle(mpq, cuda, m, n, k, a_bits, w_bits):
    """(4096 x 4096 x 128 is 512 tiles for 148 persistent CTAs: both TMEM accumulators get reused.)"""
    x = inputs.uniform_levels(15, a_bits, (m, k), a_bits)
    w = inputs.uniform_levels(15, 10 + w_bits, (n, k), w_bits)
    qa = oracle.quantize(x, 1.0, a_bits)
    qb = oracle.quantize(w, 1.0, w_bits)
    ref = oracle.gemm(qa, qb)
    a = torch.from_numpy(qa.astype(np.int8)).to(cuda)
    b = torch.from_numpy(qb.astype(np.int8)).to(cuda)
    out = torch.full((m, n), -7, dtype=torch.int32, device=cuda)
    err = torch.zeros(1, dtype=torch.int32, device=cuda)
    context.i8_gemm(a, b, out, err)
    torch.cuda.synchronize()
    assert int(err.cpu()[0]) == 0
    assert np.array_equal(out.cpu().numpy(), ref)
    # ... and the bit-plane path gives the same integers
    one = torch.ones(1, device=cuda)
    ap = mpq.encode(torch.from_numpy(x).to(cuda), one, a_bits)
    wp = mpq.encode(torch.from_numpy(w).to(cuda), one, w_bits)
    ci = torch.empty((m, n), dtype=torch.int32, device=cuda)
    mpq.gemm(ap, a_bits, wp, w_bits, m, n, k, ci, None)
    assert torch.equal(ci, out)


@pytest.mark.parametrize("m,n,k", [(128, 256, 512), (256, 512, 4096), (3072, 4096, 256)])
def test_unsigned_form_with_eq17_correction_equals_the_oracle(mpq, cuda, m, n, k):
    """8-bit codes: |q| reaches 255, so the operands are the level indices u and the store applies
    4 sum u_a u_b - 2 L_b sum u_a - 2 L_a sum u_b + k L_a L_b."""
    x = inputs.uniform_levels(16, 1, (m, k), 8)
    w = inputs.uniform_levels(16, 2, (n, k), 8)
    qa, qb = oracle.quantize(x, 1.0, 8), oracle.quantize(w, 1.0, 8)
    ref = oracle.gemm(qa, qb)
    ua = torch.from_numpy(oracle.levels(qa, 8).astype(np.uint8)).to(cuda)
    ub = torch.from_numpy(oracle.levels(qb, 8).astype(np.uint8)).to(cuda)
    sa, sb = context.row_sums_u8(ua), context.row_sums_u8(ub)
    assert np.array_equal(sa.cpu().numpy(), oracle.levels(qa, 8).sum(axis=1))
    out = torch.full((m, n), -7, dtype=torch.int32, device=cuda)
    err = torch.zeros(1, dtype=torch.int32, device=cuda)
    context.i8_gemm(ua, ub, out, err, unsigned_levels=(255, 255), sums=(sa, sb))
    torch.cuda.synchronize()
    assert int(err.cpu()[0]) == 0
    assert np.array_equal(out.cpu().numpy(), ref)
    assert np.abs(ref).max() > 127 * 127                     # levels beyond the int8 range took part


def test_shapes_outside_the_tile_grid_are_refused(cuda):
    a = torch.zeros((256, 128), dtype=torch.int8, device=cuda)
    out = torch.zeros((128, 256), dtype=torch.int32, device=cuda)
    err = torch.zeros(1, dtype=torch.int32, device=cuda)
    L = context.lib()
    assert L.mpqctx_i8_gemm(a.data_ptr(), a.data_ptr(), 100, 256, 128, out.data_ptr(), 0, None, None, 0, 0, err.data_ptr(), None) == 2
    assert L.mpqctx_i8_gemm(a.data_ptr(), a.data_ptr(), 128, 128, 128, out.data_ptr(), 0, None, None, 0, 0, err.data_ptr(), None) == 2
    assert L.mpqctx_i8_gemm(a.data_ptr(), a.data_ptr(), 128, 256, 96, out.data_ptr(), 0, None, None, 0, 0, err.data_ptr(), None) == 2
    assert L.mpqctx_i8_gemm(None, a.data_ptr(), 128, 256, 128, out.data_ptr(), 0, None, None, 0, 0, err.data_ptr(), None) == 1
    assert L.mpqctx_i8_gemm(a.data_ptr(), a.data_ptr(), 128, 256, 128, out.data_ptr(), 1, None, None, 3, 3, err.data_ptr(), None) == 1
