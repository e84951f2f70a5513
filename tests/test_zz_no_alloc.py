"""mpq_linear_static: the fully-connected layer for callers that cannot allocate device memory
(a plug-in inside a framework that owns the memory pool, a service past its start-up phase, a
program with no allocator to lend a workspace).  Its scratch is a buffer built into the library.

Collected last on purpose: a run that stops at the first failure has then already run every
other test.  Checked through the C ABI against mpq_linear (caller-provided workspace) AND
against the CPU oracle, on two calls in a row that share the built-in buffer: int32 bit-exact,
fp32 within 1e-5 relative; then at the edge of the buffer: the largest problem it takes and the
smallest it refuses.
"""
import numpy as np
import pytest
import torch

import oracle
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
    # ... and both agree with the oracle's layer on the same inputs
    acc, out, _, _ = oracle.linear(x, w, a_bits, w_bits, w_per_row=bool(w_mode), a_act=a_act)
    assert np.array_equal(got_i.cpu().numpy(), acc)
    assert rel_close(got_f.cpu().numpy(), out, 1e-5)
    assert np.unique(acc).size > 8                          # a real result, not a constant


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


def test_linear_static_at_the_edge_of_its_buffer(mpq, cuda):
    """The largest layer whose scratch still fits the built-in buffer runs and matches the oracle;
    one more weight row no longer fits and is refused.  W8A8 with k = 2048: a weight row costs
    8 planes x 64 words x 4 bytes = 2 KiB of planes plus 4 bytes of range."""
    a_bits = w_bits = 8
    m, k = 32, 2048
    fits = lambda n: mpq.linear_workspace(m, n, k, a_bits, w_bits) <= mpq.LINEAR_STATIC_BYTES
    lo, hi = 1, 1 << 20
    assert fits(lo) and not fits(hi)
    while hi - lo > 1:                                        # the workspace grows with n: bisect the edge
        mid = (lo + hi) // 2
        lo, hi = (mid, hi) if fits(mid) else (lo, mid)
    n_fit, n_over = lo, hi
    assert 7000 < n_fit < 8192
    x = inputs.uniform_levels(7, 1, (m, k), a_bits)
    w = inputs.uniform_levels(7, 2, (n_over, k), w_bits)
    xd, wd = torch.from_numpy(x).to(cuda), torch.from_numpy(w).to(cuda)
    out = torch.full((m, n_over), -7, dtype=torch.int32, device=cuda)
    L = mpq.lib()
    rc = L.mpq_linear_static(xd.data_ptr(), wd.data_ptr(), m, n_over, k, a_bits, w_bits, 0, 1, out.data_ptr(), None, None)
    assert rc == 8                                            # smallest refused size
    torch.cuda.synchronize()
    assert int((out != -7).sum()) == 0                        # ... and nothing was written
    got = torch.full((m, n_fit), -7, dtype=torch.int32, device=cuda)
    mpq.linear_static(xd, wd[:n_fit].contiguous(), a_bits, w_bits, mpq.ACT_HTANH, mpq.SCALE_PER_ROW, got, None)
    torch.cuda.synchronize()
    acc, _, _, _ = oracle.linear(x, w[:n_fit], a_bits, w_bits, w_per_row=True)
    assert np.array_equal(got.cpu().numpy(), acc)             # largest accepted size
