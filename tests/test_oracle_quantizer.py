"""Pins for the oracle's range and quantizer steps (CPU only).

Each test checks ``oracle`` against something the paper or the mathematics
fixes, never against the oracle's own formula: the printed Table 2, Eq. 15 in
exact rationals, the trigonometric encoders of Eq. 11, the odd-integer level
set of Eq. 20, the affine map of Eq. 16 and the HReLU special case.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle


def _read_table2(golden_dir):
    rows = []
    with open(os.path.join(golden_dir, "table2_states.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            frac, hi, lo = line.split()
            rows.append((Fraction(frac), int(hi), int(lo)))
    return rows


def test_table2_states(golden_dir):
    """Table 2: the four 2-bit levels and their {high, low} states; x = x1 + 2 x2; alpha = 3."""
    rows = _read_table2(golden_dir)
    assert len(rows) == 4
    x = np.array([float(fr) for fr, _, _ in rows], dtype=np.float32)
    q = oracle.quantize(x, 1.0, 2)
    u = oracle.levels(q, 2)
    for (fr, hi, lo), qi, ui in zip(rows, q.tolist(), u.tolist()):
        assert qi == lo + 2 * hi                      # x = x1 + 2 x2 on the encoded integers
        assert Fraction(qi, 3) == fr                  # alpha = 3 between number and state
        assert ((ui >> 1) & 1) * 2 - 1 == hi          # bit 1 <-> +1, bit 0 <-> -1
        assert (ui & 1) * 2 - 1 == lo


def _eq15_round_half_up(x: Fraction, k: int) -> Fraction:
    """Eq. 15 evaluated exactly, with <.> = round half up."""
    L = 2 ** k - 1
    t = L * (x + 1) / 2
    u = math.floor(t + Fraction(1, 2))
    return 2 * (Fraction(u, L) - Fraction(1, 2))


@pytest.mark.parametrize("bits", range(1, 9))
def test_eq15_exact_rationals(bits):
    """q / (2^k - 1) equals q_k(x) of Eq. 15 on a dyadic grid (exact in fp32), ties included."""
    L = 2 ** bits - 1
    grid = [Fraction(i, 1024) for i in range(-1024, 1025)]
    x = np.array([float(g) for g in grid], dtype=np.float32)
    q = oracle.quantize(x, 1.0, bits)
    for g, qi in zip(grid, q.tolist()):
        assert Fraction(qi, L) == _eq15_round_half_up(g, bits), (g, qi)
    # x = 0 is a tie at every bit-width; round half up sends it to the level just above zero
    assert oracle.quantize(np.zeros(1, np.float32), 1.0, bits)[0] == 1


@pytest.mark.parametrize("bits", range(1, 9))
def test_eq15_near_thresholds(bits):
    """Just below / above every level midpoint the code steps by exactly one level."""
    L = 2 ** bits - 1
    for j in range(-(2 ** (bits - 1)) + 1, 2 ** (bits - 1)):
        thr = 2.0 * j / L                              # L*x/2 = j
        lo = np.float32(thr) - np.float32(1e-4)
        hi = np.float32(thr) + np.float32(1e-4)
        q = oracle.quantize(np.array([lo, hi], np.float32), 1.0, bits).tolist()
        assert q == [2 * (j - 1 + 2 ** (bits - 1)) - L, 2 * (j + 2 ** (bits - 1)) - L]


def test_eq11_two_bit_trig_encoders():
    """Eq. 11: phi_2^2 = sign(sin(3/4 pi x)) is the high bit, phi_2^1 = sign(-sin(3/2 pi x)) the low bit."""
    xs = np.linspace(-1.0, 1.0, 4001)
    keep = np.ones_like(xs, dtype=bool)
    for thr in (-2 / 3, 0.0, 2 / 3, -1.0, 1.0):        # zeros of the sines: sign undefined there
        keep &= np.abs(xs - thr) > 1e-3
    xs = xs[keep].astype(np.float32)
    u = oracle.levels(oracle.quantize(xs, 1.0, 2), 2)
    hi = np.sign(np.sin(0.75 * np.pi * xs.astype(np.float64)))
    lo = np.sign(-np.sin(1.5 * np.pi * xs.astype(np.float64)))
    assert np.array_equal(((u >> 1) & 1) * 2 - 1, hi.astype(np.int64))
    assert np.array_equal((u & 1) * 2 - 1, lo.astype(np.int64))


@pytest.mark.parametrize("bits", [1, 3, 4])
def test_trig_encoders_general_bits(bits):
    """The periodic-encoder family continued to other widths: the top bit has half a period
    on [-1, 1] scaled by L/2^b, each lower bit doubles the frequency (Fig. 2's description)."""
    L = 2 ** bits - 1
    xs = np.linspace(-0.999, 0.999, 5003)
    thr = np.array([2.0 * j / L for j in range(-(2 ** (bits - 1)) + 1, 2 ** (bits - 1))])
    keep = np.min(np.abs(xs[:, None] - thr[None, :]), axis=1) > 1e-3
    xs = xs[keep].astype(np.float32)
    u = oracle.levels(oracle.quantize(xs, 1.0, bits), bits)
    x64 = xs.astype(np.float64)
    top = np.sign(np.sin(L / 2 ** bits * np.pi * x64))
    assert np.array_equal(((u >> (bits - 1)) & 1) * 2 - 1, top.astype(np.int64))
    for m in range(1, bits):                           # m = 1 is the low bit
        enc = np.sign(-np.sin(L / 2 ** m * np.pi * x64))
        assert np.array_equal(((u >> (m - 1)) & 1) * 2 - 1, enc.astype(np.int64)), m


@pytest.mark.parametrize("bits", range(1, 9))
def test_eq20_odd_and_bounded(bits):
    """Eq. 20: every decoded value is an odd integer with |q| <= 2^K - 1; out-of-range inputs clamp (HTanh)."""
    rng = np.random.default_rng(7 + bits)
    x = (rng.standard_normal(20000) * 2.0).astype(np.float32)   # well beyond [-1, 1]
    x[:6] = [np.inf, -np.inf, 1e30, -1e30, 5.0, -5.0]
    q = oracle.quantize(x, 1.0, bits).astype(np.int64)
    L = 2 ** bits - 1
    assert np.all(np.abs(q) % 2 == 1)
    assert q.max() == L and q.min() == -L
    assert q[:6].tolist() == [L, -L, L, -L, L, -L]
    assert set(np.unique(q).tolist()) == set(range(-L, L + 1, 2))   # all 2^b states are reachable


@pytest.mark.parametrize("bits", [2, 3, 8])
def test_eq16_affine_map(bits):
    """Eq. 16: x^q = 2/(2^M-1) * x^{0,1} - 1 links the level index u to the quantized number q/L."""
    rng = np.random.default_rng(11)
    x = rng.uniform(-1, 1, 1000).astype(np.float32)
    q = oracle.quantize(x, 1.0, bits)
    u = oracle.levels(q, bits)
    L = 2 ** bits - 1
    for qi, ui in zip(q.tolist(), u.tolist()):
        assert Fraction(qi, L) == Fraction(2 * ui, L) - 1
        assert 0 <= ui <= L


def test_monotone_and_symmetric_levels():
    """The ladder is non-decreasing, and q(-x) = -q(x) away from the midpoints."""
    xs = np.linspace(-1.5, 1.5, 3001).astype(np.float32)
    for bits in (1, 2, 5):
        q = oracle.quantize(xs, 1.0, bits).astype(np.int64)
        assert np.all(np.diff(q) >= 0)
        L = 2 ** bits - 1
        thr = np.array([2.0 * j / L for j in range(-(2 ** (bits - 1)), 2 ** (bits - 1) + 1)])
        keep = np.min(np.abs(xs[:, None] - thr[None, :]), axis=1) > 1e-3
        assert np.array_equal(q[keep], -q[::-1][keep])


def test_scale_is_division_then_clamp():
    """A max-abs scale s reduces to the paper's fixed range: quantize(x, s) == quantize(x/s, 1)
    whenever x/s is exact (power-of-two s)."""
    rng = np.random.default_rng(3)
    x = rng.standard_normal(5000).astype(np.float32)
    for s in (0.5, 2.0, 8.0):
        for bits in (2, 4):
            a = oracle.quantize(x, s, bits)
            b = oracle.quantize((x / np.float32(s)).astype(np.float32), 1.0, bits)
            assert np.array_equal(a, b)


def test_per_row_scale():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((6, 100)).astype(np.float32)
    s = np.array([0.5, 1, 2, 4, 8, 16], np.float32)
    q = oracle.quantize(x, s, 3, per_row=True)
    for r in range(6):
        assert np.array_equal(q[r], oracle.quantize(x[r], s[r], 3))


def test_degenerate_scales_and_nan():
    """A scale that is zero, negative, infinite or NaN makes 1/s := 0: every code is the level
    just above zero (q = +1).  A NaN input does the same for that element."""
    x = np.array([-3.0, -0.1, 0.0, 0.1, 3.0], np.float32)
    for s in (0.0, -1.0, np.inf, np.nan):
        assert oracle.quantize(x, s, 3).tolist() == [1] * 5
    xn = np.array([np.nan, 0.9], np.float32)
    assert oracle.quantize(xn, 1.0, 2).tolist() == [1, 3]


def test_hrelu_one_bit_gives_all_plus_one():
    """HReLU with the 1-bit encoder constrains every activation to +1 (Section 5.1, ImageNet)."""
    rng = np.random.default_rng(9)
    x = rng.standard_normal(4000).astype(np.float32)
    q = oracle.quantize(x, 1.0, 1, act=oracle.HRELU)
    assert np.all(q == 1)
    # ... and with more bits the negative side collapses onto the level just above zero
    q3 = oracle.quantize(x, 1.0, 3, act=oracle.HRELU)
    assert np.all(q3[x < 0] == 1) and q3.min() == 1
    # on the non-negative side HReLU and HTanh agree
    assert np.array_equal(q3[x >= 0], oracle.quantize(x, 1.0, 3)[x >= 0])


def test_absmax_matches_numpy():
    rng = np.random.default_rng(13)
    x = rng.standard_normal((37, 211)).astype(np.float32)
    x[3, 5] = np.nan                                    # ignored
    ref = np.nanmax(np.abs(x))
    assert oracle.absmax(x)[0] == ref
    assert np.array_equal(oracle.absmax(x, per_row=True), np.nanmax(np.abs(x), axis=1))
    assert oracle.absmax(x, act=oracle.HRELU)[0] == np.nanmax(np.maximum(x, 0))
    assert oracle.absmax(-np.abs(x), act=oracle.HRELU)[0] == 0.0


def _eq15_level_of(x: Fraction, bits: int) -> int:
    """Odd integer of Eq. 15 (round half up) for a real x, with the HTanh clamp to [-1, 1] first."""
    L = 2 ** bits - 1
    x = max(Fraction(-1), min(Fraction(1), x))
    u = math.floor(L * (x + 1) / 2 + Fraction(1, 2))
    return 2 * min(u, L) - L


@pytest.mark.parametrize("s", [0.37, 3.7])
@pytest.mark.parametrize("bits", [1, 2, 3, 5, 8])
def test_eq15_of_x_over_s_for_ranges_that_are_not_powers_of_two(s, bits):
    """With a range s that is not a power of two the code is Eq. 15 of the real quotient x/s
    (exact rationals of the float32 inputs), for every input that is not within a few fp32
    roundings of a level boundary (there the two rounded multiplies may legitimately decide
    either way)."""
    rng = np.random.default_rng(61 + bits)
    s32 = np.float32(s)
    x = (rng.uniform(-1.3, 1.3, 6000) * s).astype(np.float32)
    L = 2 ** bits - 1
    q = oracle.quantize(x, s32, bits).tolist()
    checked = 0
    for xi, qi in zip(x.tolist(), q):
        t = Fraction(xi) / Fraction(float(s32)) * L / 2          # level boundaries are the integers of t
        if abs(t - round(t)) <= 8 * Fraction(2) ** -23 * max(1, abs(t)):
            continue
        assert qi == _eq15_level_of(Fraction(xi) / Fraction(float(s32)), bits), (xi, qi)
        checked += 1
    assert checked > 5900


def test_trig_encoder_reproduces_table2(golden_dir):
    """The trigonometric form (Eq. 11) sends Table 2's four printed levels to their printed states."""
    rows = _read_table2(golden_dir)
    x = np.array([float(fr) for fr, _, _ in rows], dtype=np.float32)
    u = oracle.levels(oracle.quantize_trig(x, 1.0, 2), 2)
    for (fr, hi, lo), ui in zip(rows, u.tolist()):
        assert ((ui >> 1) & 1) * 2 - 1 == hi and (ui & 1) * 2 - 1 == lo


@pytest.mark.parametrize("bits", range(1, 9))
@pytest.mark.parametrize("act", [oracle.HTANH, oracle.HRELU])
def test_trig_encoder_equals_eq15_away_from_level_boundaries(bits, act):
    """Bit by bit the sine encoders spell the level index of Eq. 15 (exact rationals, round half up)
    for every input that is not within a few roundings of a level boundary; at x = 0, a zero of every
    sine, each sign is that of the sine just above the zero, which spells the level above zero (the
    round-half-up tie); beyond the range the code saturates."""
    rng = np.random.default_rng(83 + bits)
    s32 = np.float32(1.7)
    x = (rng.uniform(-1.4, 1.4, 5000) * 1.7).astype(np.float32)
    x[:3] = [0.0, 40.0, -40.0]
    L = 2 ** bits - 1
    q = oracle.quantize_trig(x, s32, bits, act=act).tolist()
    checked = 0
    for xi, qi in zip(x.tolist(), q):
        y = Fraction(xi) / Fraction(float(s32))
        if act == oracle.HRELU:
            y = max(y, Fraction(0))
        t = y * L / 2
        if y != 0 and abs(t) < 2 ** (bits - 1) and abs(t - round(t)) <= 8 * Fraction(2) ** -23 * max(1, abs(t)):
            continue                                    # y == 0 is kept: the tie itself is pinned
        assert qi == _eq15_level_of(y, bits), (xi, qi)
        checked += 1
    assert checked > 4900
    assert q[0] == 1 and q[1] == L and q[2] == (1 if act == oracle.HRELU else -L)


def test_trig_encoder_special_values():
    """NaN takes the tie's level; an unusable range makes every code the level above zero."""
    x = np.array([np.nan, -0.9, 0.9], np.float32)
    assert oracle.quantize_trig(x, 1.0, 3).tolist() == [1, -7, 7]
    for s in (0.0, -2.0, np.inf, np.nan):
        assert oracle.quantize_trig(x, s, 3).tolist() == [1, 1, 1]
    big = np.array([np.inf, -np.inf, 3e38], np.float32)
    assert oracle.quantize_trig(big, 1.0, 2).tolist() == [3, -3, 3]
