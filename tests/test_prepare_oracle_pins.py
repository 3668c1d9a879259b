"""Pins of the oracle's Q/K producer (RMS normalisation + rotary embedding + one bf16 rounding):
hand examples with exactly representable results, rounding cases that a detour through fp32
gets wrong, invariants of the normalisation and of the rotation."""
import numpy as np
import torch

import oracle


def bf16_bits(x):
    return torch.tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def bits_to_f64(b):
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def test_hand_example_norm_gain_rotation():
    # a row of ones has RMS 1, so y = gain; the pair (2, 4) turned by the angle with cos 0.6, sin 0.8 is (-2, 4)
    D = 8
    x = bf16_bits(np.ones((1, 1, D)))
    gain = np.array([2, 4, 1, 0, 3, 3, 0.5, -0.5], dtype=np.float32)
    rot = np.zeros((1, D // 2, 2), dtype=np.float32)
    rot[0, :, 0] = [0.6, 1.0, 0.0, -1.0]
    rot[0, :, 1] = [0.8, 0.0, 1.0, 0.0]
    out = bits_to_f64(oracle.qk_prepare(x, gain, rot, 0.0))[0, 0]
    np.testing.assert_array_equal(out, [-2.0, 4.0, 1.0, 0.0, -3.0, 3.0, -0.5, 0.5])
    # a wrong divisor (sum instead of mean) or a missing square root would change this one
    x = bf16_bits(np.array([[[3.0, 4.0, 0.0, 0.0]]]))             # mean square 6.25, RMS 2.5
    out = bits_to_f64(oracle.qk_prepare(x, np.ones(4, np.float32), None, 0.0))[0, 0]
    np.testing.assert_array_equal(out, bits_to_f64(bf16_bits([1.2, 1.6, 0.0, 0.0])))
    out = bits_to_f64(oracle.qk_prepare(x, np.ones(4, np.float32), None, 2.75))[0, 0]   # 6.25 + 2.75 = 9
    np.testing.assert_array_equal(out, [1.0, 1.3359375, 0.0, 0.0])             # 4/3 -> 1 + 43/128


def test_rounding_is_direct_nearest_even():
    # rows of +-1 have RMS 1: out = gain rounded to bf16 (8 significant bits)
    D = 8
    x = bf16_bits(np.ones((1, 1, D)))
    g = np.array([1 + 2.0 ** -8,                 # tie between 1 and 1 + 2^-7: even mantissa wins -> 1
                  1 + 3 * 2.0 ** -8,             # tie between 1 + 2^-7 and 1 + 2^-6 -> 1 + 2^-6
                  1 + 2.0 ** -8 + 2.0 ** -20,    # just above the tie -> 1 + 2^-7
                  1 + 2.0 ** -8 - 2.0 ** -20,    # just below -> 1
                  255.5, 1e-30, 0.0, -1 - 2.0 ** -8], dtype=np.float32)
    out = bits_to_f64(oracle.qk_prepare(x, g, None, 0.0))[0, 0]
    np.testing.assert_array_equal(out[:5], [1.0, 1 + 2.0 ** -6, 1 + 2.0 ** -7, 1.0, 256.0])
    assert abs(out[5] / 1e-30 - 1) < 2.0 ** -8                               # small exponents survive
    assert out[6] == 0.0 and out[7] == -1.0
    # fp64 products that fp32 cannot hold: y = x * r * gain with r irrational; the result must be the
    # bf16 neighbour nearest to the exact value (checked with exact rational arithmetic)
    from fractions import Fraction
    rng = np.random.default_rng(0)
    xs = bf16_bits(rng.standard_normal((1, 4, D)))
    gain = rng.uniform(0.5, 2.0, D).astype(np.float32)
    got = oracle.qk_prepare(xs, gain, None, 0.0)[0]
    xv = bits_to_f64(xs)[0]
    for n in range(4):
        ms = sum(Fraction(v) ** 2 for v in xv[n]) / D
        for d in range(D):
            # |z| = |x g| / sqrt(ms): compare squares to stay rational
            lo, hi = sorted([bits_to_f64(np.array([got[n, d] - 1], np.uint16))[0], bits_to_f64(np.array([got[n, d] + 1], np.uint16))[0]], key=abs)
            z2 = (Fraction(xv[n, d]) * Fraction(float(gain[d]))) ** 2 / ms
            g0 = Fraction(bits_to_f64(np.array([got[n, d]], np.uint16))[0])
            half_lo, half_hi = (Fraction(lo) + g0) / 2, (Fraction(hi) + g0) / 2
            assert half_lo ** 2 <= z2 <= half_hi ** 2 or half_hi ** 2 <= z2 <= half_lo ** 2


def test_normalisation_and_rotation_invariants():
    rng = np.random.default_rng(1)
    H, N, D = 2, 37, 64
    x = bf16_bits(rng.standard_normal((H, N, D)) * 3.0)
    ones = np.ones(D, np.float32)
    base = oracle.qk_prepare(x, ones, None, 0.0)
    # unit RMS per token (up to the bf16 rounding of the outputs)
    rms = np.sqrt((bits_to_f64(base) ** 2).mean(axis=-1))
    assert np.abs(rms - 1).max() < 2.0 ** -8
    # scaling the input by a power of two changes nothing when eps = 0
    x4 = bf16_bits(bits_to_f64(x) * 4.0)
    np.testing.assert_array_equal(oracle.qk_prepare(x4, ones, None, 0.0), base)
    # eps matters: a large eps shrinks every output
    assert (np.abs(bits_to_f64(oracle.qk_prepare(x, ones, None, 100.0))) <= np.abs(bits_to_f64(base))).all()
    # quarter turn: (y0, y1) -> (-y1, y0) exactly; half turn: sign flip; zero angle: identity
    def table(c, s):
        t = np.empty((N, D // 2, 2), np.float32)
        t[..., 0], t[..., 1] = c, s
        return t
    b = bits_to_f64(base)
    q = bits_to_f64(oracle.qk_prepare(x, ones, table(0.0, 1.0), 0.0))
    np.testing.assert_array_equal(q[..., 0::2], -b[..., 1::2])
    np.testing.assert_array_equal(q[..., 1::2], b[..., 0::2])
    np.testing.assert_array_equal(bits_to_f64(oracle.qk_prepare(x, ones, table(-1.0, 0.0), 0.0)), -b)
    np.testing.assert_array_equal(oracle.qk_prepare(x, ones, table(1.0, 0.0), 0.0), base)
    # a rotation keeps the length of every pair (up to the output rounding), token-dependent angles included
    ang = rng.uniform(0, 2 * np.pi, (N, D // 2))
    t = np.stack([np.cos(ang), np.sin(ang)], axis=-1).astype(np.float32)
    r = bits_to_f64(oracle.qk_prepare(x, ones, t, 0.0))
    len_b = np.hypot(b[..., 0::2], b[..., 1::2])
    len_r = np.hypot(r[..., 0::2], r[..., 1::2])
    assert np.abs(len_r - len_b).max() < 2.0 ** -6 * max(1.0, len_b.max())
    # the gain is applied per channel before the rotation: gain on one channel of a pair only
    g = ones.copy()
    g[0] = 0.0
    z = bits_to_f64(oracle.qk_prepare(x, g, table(0.0, 1.0), 0.0))
    np.testing.assert_array_equal(z[..., 1], 0.0 * b[..., 0])          # z1 = y0 = 0
    np.testing.assert_array_equal(z[..., 0], -b[..., 1])
