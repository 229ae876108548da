"""Pins of the oracle's root-mean-square normalisation (the producer of the activations of two
of a decoder layer's four linears) against exact rational arithmetic, closed forms and the
invariances the definition has."""
from fractions import Fraction

import numpy as np

import gen
import oracle
from helpers import bits_to_f32, f32_to_bf16_bits


def _frac_of_f32(v) -> Fraction:
    return Fraction(float(np.float32(v)))


def _round_fraction_to_f32(q: Fraction) -> np.float32:
    """Nearest fp32 (ties to even) of a positive or negative rational, by exact arithmetic."""
    if q == 0:
        return np.float32(0.0)
    sign = -1 if q < 0 else 1
    a = abs(q)
    e = 0
    while a >= 2:
        a /= 2
        e += 1
    while a < 1:
        a *= 2
        e -= 1
    scaled = a * (1 << 23)                      # in [2^23, 2^24)
    fl = scaled.numerator // scaled.denominator
    rem = scaled - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return np.float32(sign * float(Fraction(fl, 1 << 23) * Fraction(2) ** e))


def _bf16_of_f32_exact(v: np.float32) -> int:
    """bf16 bits (ties to even) of an fp32 value, from its bit pattern."""
    u = int(np.float32(v).view(np.uint32))
    low = u & 0xFFFF
    hi = u >> 16
    if low > 0x8000 or (low == 0x8000 and (hi & 1)):
        hi += 1
    return hi & 0xFFFF


def test_rmsnorm_matches_exact_rational_arithmetic():
    """Every step re-derived with Fractions on a small case: the mean of squares exactly, r as THE
    fp32 value nearest to 1/sqrt(ms + eps) (checked by squaring the two half-way points), both
    products and both roundings to bf16."""
    M, K = 6, 96
    eps = 1e-5
    xb = gen.bf16_bits(gen.activations(M, K, seed=7, outlier_fraction=0.05, outlier_scale=20.0))
    gb = gen.bf16_bits(1.0 + 0.25 * gen.weights(1, K, seed=8, std=1.0)).reshape(K)
    y, r, amb = oracle.rmsnorm(xb, gb, eps)
    assert not amb.any()
    x = bits_to_f32(xb)
    g = bits_to_f32(gb)
    eps_q = _frac_of_f32(eps)
    for m in range(M):
        ms = sum(_frac_of_f32(v) ** 2 for v in x[m]) / K
        target = ms + eps_q                      # r must be the fp32 nearest to target^(-1/2)
        rq = _frac_of_f32(r[m])
        up = _frac_of_f32(np.nextafter(r[m], np.float32(np.inf)))
        dn = _frac_of_f32(np.nextafter(r[m], np.float32(-np.inf)))
        assert ((rq + up) / 2) ** 2 * target > 1 > ((rq + dn) / 2) ** 2 * target
        for j in range(K):
            t32 = _round_fraction_to_f32(_frac_of_f32(x[m, j]) * rq)
            tb = _bf16_of_f32_exact(t32)
            tq = _frac_of_f32(bits_to_f32(np.array([tb], dtype=np.uint16))[0])
            y32 = _round_fraction_to_f32(tq * _frac_of_f32(g[j]))
            assert int(y[m, j]) == _bf16_of_f32_exact(y32), (m, j)


def test_rmsnorm_closed_forms():
    K = 64
    one = f32_to_bf16_bits(np.ones(K, dtype=np.float32))
    # a constant row without eps: every output is exactly +-1 (times gamma)
    for c in (0.5, -3.0, 1024.0):
        xb = f32_to_bf16_bits(np.full((1, K), c, dtype=np.float32))
        y, r, _ = oracle.rmsnorm(xb, one, 0.0)
        assert np.all(bits_to_f32(y) == np.sign(c))
    gb = f32_to_bf16_bits(np.linspace(-2.0, 2.0, K).astype(np.float32))
    xb = f32_to_bf16_bits(np.full((1, K), 4.0, dtype=np.float32))
    y, _, _ = oracle.rmsnorm(xb, gb, 0.0)
    assert np.array_equal(y[0], gb)              # t = 1 exactly, so y = gamma
    # (3, 4) repeated: mean of squares 12.5, r = fp32(1/sqrt(12.5))
    xb = f32_to_bf16_bits(np.tile(np.array([3.0, 4.0], dtype=np.float32), K // 2)[None, :])
    y, r, _ = oracle.rmsnorm(xb, one, 0.0)
    assert r[0] == np.float32(1.0 / np.sqrt(12.5))
    assert np.array_equal(y[0, :2], f32_to_bf16_bits(np.array([3.0, 4.0], dtype=np.float32) * r[0]))
    # a zero row: r = 1/sqrt(eps), outputs stay zero
    y, r, _ = oracle.rmsnorm(np.zeros((1, K), dtype=np.uint16), one, 1e-6)
    assert not y.any() and r[0] == np.float32(1.0 / np.sqrt(float(np.float32(1e-6))))


def test_rmsnorm_invariances():
    """Without eps the output does not change under a power-of-two rescaling of the row (r scales
    by the exact inverse) and flips sign with the input; the mean square of the output is 1 up to
    the bf16 roundings."""
    M, K = 16, 512
    xb = gen.bf16_bits(gen.activations(M, K, seed=11, outlier_fraction=0.02, outlier_scale=30.0))
    gb = f32_to_bf16_bits(np.ones(K, dtype=np.float32))
    y, r, amb = oracle.rmsnorm(xb, gb, 0.0)
    assert not amb.any()
    x = bits_to_f32(xb)
    y8, r8, _ = oracle.rmsnorm(f32_to_bf16_bits(x * np.float32(8.0)), gb, 0.0)
    assert np.array_equal(y, y8) and np.array_equal(r8 * np.float32(8.0), r)
    yn, _, _ = oracle.rmsnorm(xb ^ np.uint16(0x8000), gb, 0.0)
    assert np.array_equal(yn, y ^ np.uint16(0x8000))
    ms_out = np.mean(bits_to_f32(y).astype(np.float64) ** 2, axis=1)
    assert np.all(np.abs(ms_out - 1.0) < 2e-2)


def test_rmsnorm_encode_is_the_encode_of_the_normalised_row():
    M, K, b, k = 8, 512, 64, 8
    xb = gen.bf16_bits(gen.activations(M, K, seed=13, outlier_fraction=0.02, outlier_scale=30.0))
    gb = gen.bf16_bits(1.0 + 0.1 * gen.weights(1, K, seed=14, std=1.0)).reshape(K)
    pos = oracle.calib_positions(b, k, gen.bf16_bits(gen.calibration_batch(64, K, seed=13, outlier_fraction=0.02, outlier_scale=30.0)))
    enc, y = oracle.rmsnorm_encode(b, k, xb, gb, 1e-5, pos)
    ref = oracle.encode(b, k, y, pos)
    assert np.array_equal(enc.dq4, ref.dq4) and np.array_equal(enc.vals, ref.vals)
    # the row maximum of a normalised row maps to +-127
    assert np.all(np.abs(enc.vals).reshape(M, -1).max(axis=1) <= 127)
