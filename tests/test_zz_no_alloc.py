"""mpq_linear_static: the fully-connected layer for callers that cannot allocate device memory
(a plug-in inside a framework that owns the memory pool, a service past its start-up phase, a
program with no allocator to lend a workspace).  Its scratch is a buffer built into the library.

Collected last on purpose: a run that stops at the first failure has then already run every
other test.  Checked against mpq_linear (caller-provided workspace) through the C ABI, on two
calls in a row that share the built-in buffer: int32 bit-exact, fp32 within 1e-5 relative.
"""
import numpy as np
import pytest
import torch

from paper_1905_13389_b200 import inputs
from tests._util import rel_close

pytestmark = pytest.mark.gpu


def _layer_both_ways(mpq, cuda, x, w, a_bits, w_bits, a_act, w_mode):
    m, n = x.shape[0], w.shape[0]
    xd = torch.from_numpy(x).to(cuda)
    wd = torch.from_numpy(w).to(cuda)
    ref_i = torch.empty((m, n), dtype=torch.int32, device=cuda)
    ref_f = torch.empty((m, n), dtype=torch.float32, device=cuda)
    mpq.linear(xd, wd, a_bits, w_bits, a_act, w_mode, ref_i, ref_f)
    # poison the outputs so that an entry point that writes nothing cannot pass
    got_i = torch.full((m, n), -7, dtype=torch.int32, device=cuda)
    got_f = torch.full((m, n), float("nan"), dtype=torch.float32, device=cuda)
    mpq.linear_static(xd, wd, a_bits, w_bits, a_act, w_mode, got_i, got_f)
    torch.cuda.synchronize()
    assert np.array_equal(got_i.cpu().numpy(), ref_i.cpu().numpy())
    assert rel_close(got_f.cpu().numpy(), ref_f.cpu().numpy(), 1e-5)
    assert np.unique(ref_i.cpu().numpy()).size > 8          # a real result, not a constant


def test_linear_static_matches_linear_on_two_calls_in_a_row(mpq, cuda):
    # first call: the 64 x 64 x 512 W2A2 layer; second call: a smaller, ragged W3A4 layer with
    # per-row weight ranges, so stale contents of the shared buffer from call one would show
    c = inputs.config1()
    _layer_both_ways(mpq, cuda, c["x"], c["w"], 2, 2, mpq.ACT_HTANH, mpq.SCALE_PER_TENSOR)
    x = inputs.uniform_levels(6, 1, (19, 333), 3)
    w = inputs.uniform_levels(6, 2, (45, 333), 4)
    _layer_both_ways(mpq, cuda, x, w, 3, 4, mpq.ACT_HRELU, mpq.SCALE_PER_ROW)


def test_linear_static_rejects_problems_beyond_its_buffer(mpq, cuda):
    """Sizes whose scratch exceeds MPQ_LINEAR_STATIC_BYTES are refused with their own status,
    before anything is launched (the tensors here are never read)."""
    m, n, k = 64, 8192, 16384                                  # W8 planes alone: 8 * 8192 * 2 KiB = 128 MiB
    assert mpq.linear_workspace(m, n, k, 8, 8) > mpq.LINEAR_STATIC_BYTES
    x = torch.empty((m, k), dtype=torch.float32, device=cuda)
    w = torch.empty((1, k), dtype=torch.float32, device=cuda).expand(n, k)   # no real 512 MiB tensor needed
    out = torch.empty((m, n), dtype=torch.int32, device=cuda)
    rc = mpq.lib().mpq_linear_static(x.data_ptr(), w.data_ptr(), m, n, k, 8, 8, 0, 0, out.data_ptr(), None, None)
    assert rc == 8 and "MPQ_LINEAR_STATIC_BYTES" in mpq.status_string(rc)
