"""Pins of the oracle's Cache-Reuse data path (Sec. 3.2 "Level-2: Cache-Reuse"): exact rational
arithmetic with a rounding routine written here from the IEEE definition (round to nearest, ties
to even, first to 24 then to 8 significant bits), closed forms, and the action semantics."""
from fractions import Fraction

import numpy as np
import torch

import oracle


def bf16_bits(x: np.ndarray) -> np.ndarray:
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def bits_to_fraction(b: int) -> Fraction:
    sign = -1 if b & 0x8000 else 1
    e, m = (b >> 7) & 0xFF, b & 0x7F
    assert 0 < e < 255                                     # normal numbers only in these tests
    return sign * Fraction(128 + m, 128) * Fraction(2) ** (e - 127)


def round_fraction(v: Fraction, bits: int) -> Fraction:
    """Round to `bits` significant bits, nearest, ties to even (normal range assumed)."""
    if v == 0:
        return v
    s, a = (1 if v > 0 else -1), abs(v)
    e = 0
    while Fraction(2) ** (e + 1) <= a:
        e += 1
    while Fraction(2) ** e > a:
        e -= 1
    q = Fraction(2) ** (e - bits + 1)                      # spacing of representable values
    n = a / q
    lo = n.numerator // n.denominator
    rem = n - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    return s * lo * q


def fraction_to_bf16_bits(v: Fraction) -> int:
    if v == 0:
        return 0
    return int(bf16_bits(np.array([float(v)]))[0])         # v is exactly a bf16 value here


def test_sum_and_difference_against_exact_rational_arithmetic():
    rng = np.random.default_rng(5)
    # magnitudes spread over 30 binades so that fp32 rounding before the bf16 rounding matters
    mag = np.exp2(rng.uniform(-15, 15, size=(2, 400))) * rng.choice([-1.0, 1.0], size=(2, 400))
    xb, yb = bf16_bits(mag[0]), bf16_bits(mag[1])
    x, y = xb.reshape(1, -1), yb.reshape(1, -1)
    o_new, _ = oracle.cache_step(x, np.zeros_like(x), y, [1])          # o = x + delta
    _, d_new = oracle.cache_step(x, y, np.zeros_like(x), [2])          # delta = o - x
    for i in range(x.shape[1]):
        fx, fy = bits_to_fraction(int(xb[i])), bits_to_fraction(int(yb[i]))
        want_sum = round_fraction(round_fraction(fx + fy, 24), 8)
        want_dif = round_fraction(round_fraction(fy - fx, 24), 8)
        assert int(o_new[0, i]) == fraction_to_bf16_bits(want_sum), i
        assert int(d_new[0, i]) == fraction_to_bf16_bits(want_dif), i


def test_refresh_then_reuse_returns_the_output_when_the_residual_is_exact():
    rng = np.random.default_rng(6)
    x = rng.integers(-60, 60, size=(3, 64)).astype(np.float32)          # small integers: o - x is exact in bf16
    o = x + rng.integers(-60, 60, size=(3, 64)).astype(np.float32)
    xb, ob = bf16_bits(x), bf16_bits(o)
    assert (oracle._bf16_bits_to_f32(xb) == x).all() and (oracle._bf16_bits_to_f32(ob) == o).all()
    _, delta = oracle.cache_step(xb, ob, np.zeros_like(xb), [2, 2, 2])
    o2, _ = oracle.cache_step(xb, np.zeros_like(xb), delta, [1, 1, 1])
    assert (o2 == ob).all()
    # zero residual: reuse returns the input itself
    o3, _ = oracle.cache_step(xb, ob, np.zeros_like(xb), [1, 1, 1])
    assert (o3 == xb).all()


def test_actions_select_the_branch_per_image():
    rng = np.random.default_rng(7)
    xb, ob, db = (bf16_bits(rng.normal(size=(3, 32))) for _ in range(3))
    o_new, d_new = oracle.cache_step(xb, ob, db, [0, 1, 2])
    assert (o_new[0] == ob[0]).all() and (d_new[0] == db[0]).all()      # skipped: untouched
    assert (d_new[1] == db[1]).all() and not (o_new[1] == ob[1]).all()  # reuse writes o only
    assert (o_new[2] == ob[2]).all() and not (d_new[2] == db[2]).all()  # attend writes delta only
