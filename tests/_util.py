"""Test-side helpers: unpacking of the packed bit-planes (independent of both implementations)."""
import numpy as np


def unpack_planes(planes: np.ndarray, k: int) -> np.ndarray:
    """planes [bits][rows][row_words] (uint32 words) -> level index u [rows][k]; also checks that
    every bit past element k-1 is zero."""
    planes = planes.view(np.uint32)
    bits, rows, rw = planes.shape
    shifts = np.arange(32, dtype=np.uint32)
    u = np.zeros((rows, rw * 32), dtype=np.int64)
    for p in range(bits):
        b = ((planes[p][:, :, None] >> shifts[None, None, :]) & 1).reshape(rows, rw * 32)
        u += b.astype(np.int64) << p
    assert not u[:, k:].any(), "padding bits must be zero"
    return u[:, :k]


def pack_levels(u: np.ndarray, bits: int, row_words: int) -> np.ndarray:
    """Level index u [rows][k] -> planes [bits][rows][row_words] uint32 (test-side packer)."""
    rows, k = u.shape
    padded = np.zeros((rows, row_words * 32), dtype=np.uint64)
    padded[:, :k] = u
    out = np.zeros((bits, rows, row_words), dtype=np.uint32)
    weights = (np.uint64(1) << np.arange(32, dtype=np.uint64))
    for p in range(bits):
        b = (padded >> np.uint64(p)) & np.uint64(1)
        out[p] = (b.reshape(rows, row_words, 32) * weights[None, None, :]).sum(axis=2).astype(np.uint32)
    return out


def rel_close(got: np.ndarray, ref: np.ndarray, rel: float = 1e-5) -> bool:
    """|g - r| <= rel * |r| element-wise; exact where r == 0."""
    got = got.astype(np.float64)
    ref = ref.astype(np.float64)
    return bool(np.all(np.abs(got - ref) <= rel * np.abs(ref)))
