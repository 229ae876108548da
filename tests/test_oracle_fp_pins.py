"""Pins of the floating-point (FP8 sparse + FP4 dense) oracle against what is fixed independently of
it: the OCP E2M1 / E4M3 value sets by enumeration, a library conversion for E4M3, exact rational
arithmetic for every rounding, brute force for the selection and the GEMM.  CPU only."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import gen
import oracle
from helpers import bits_to_f32

E2M1_MAGS = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]      # the eight magnitudes of the 4-bit format


def _acts(M, K, seed):
    return gen.bf16_bits(gen.activations(M, K, seed=seed, outlier_fraction=0.02, outlier_scale=20.0))


def _nearest_even(v: Fraction, grid):
    """Index of the grid value nearest to v (grid ascending, non-negative v), ties to the even index,
    beyond the last value: the last one."""
    if v >= grid[-1]:
        return len(grid) - 1
    best = min(range(len(grid)), key=lambda i: (abs(grid[i] - v), i % 2))
    return best


def test_value_tables_by_enumeration():
    e2, e4 = oracle.fp_tables()
    assert e2[:8].tolist() == E2M1_MAGS and e2[8:].tolist() == [-x for x in E2M1_MAGS]
    # E4M3: every finite code against the library's own decoding of the byte
    codes = torch.arange(256, dtype=torch.uint8)
    lib = codes.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    finite = ~np.isnan(lib)
    assert finite.sum() == 254 and np.isnan(e4[0x7F]) and np.isnan(e4[0xFF])
    assert np.array_equal(e4[finite], lib[finite])
    assert e4[0x7E] == 448.0 and e4[0x01] == 2.0 ** -9 and e4[0x08] == 2.0 ** -6


def test_e4m3_rounding_is_the_library_conversion_and_exact():
    rng = np.random.default_rng(0)
    v = np.concatenate([rng.standard_normal(20000) * rng.choice([1e-3, 0.1, 3.0, 100.0], 20000), [0.0, 448.0, -448.0, 2.0 ** -10, 3 * 2.0 ** -10]])
    v = v[np.abs(v) <= 448.0].astype(np.float32)
    got = oracle.fp_round("e4m3", v.astype(np.float64))
    lib = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    _, e4 = oracle.fp_tables()
    assert np.array_equal(e4[got], e4[lib])                      # same values (signs of zero aside)
    # exact ties and saturation, against rationals
    grid = [Fraction(float(x)) for x in e4[:0x7F]]
    for i in range(0, 0x7E):
        mid = (grid[i] + grid[i + 1]) / 2
        code = int(oracle.fp_round("e4m3", np.array([float(mid)]))[0])
        assert code == (i if i % 2 == 0 else i + 1)
    assert int(oracle.fp_round("e4m3", np.array([1e9]))[0]) == 0x7E and int(oracle.fp_round("e4m3", np.array([-500.0]))[0]) == 0xFE


def test_e2m1_rounding_against_exact_rationals():
    grid = [Fraction(x) for x in E2M1_MAGS]
    rng = np.random.default_rng(1)
    vals = np.concatenate([rng.uniform(-7.5, 7.5, 5000), [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0, 6.5, 100.0, -0.25, -5.0]])
    got = oracle.fp_round("e2m1", vals)
    for v, c in zip(vals, got):
        want = _nearest_even(abs(Fraction(float(v))), grid) | (8 if v < 0 else 0)
        assert int(c) == want, (v, c, want)
    # the tie cases spelled out: 0.25 -> 0, 0.75 -> 1, 1.25 -> 1, 1.75 -> 2, 2.5 -> 2, 3.5 -> 4, 5 -> 4
    assert [E2M1_MAGS[int(c)] for c in oracle.fp_round("e2m1", np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]))] == [0, 1, 1, 2, 2, 4, 4]


def _unpack4(packed):
    lo, hi = packed & 0xF, packed >> 4
    return np.stack([lo, hi], axis=-1).reshape(*packed.shape[:-1], packed.shape[-1] * 2)


@pytest.mark.parametrize("b,k,static", [(32, 4, False), (64, 8, True), (128, 16, False)])
def test_encode_against_exact_rationals_and_invariants(b, k, static):
    M, K = 6, 256
    x = _acts(M, K, seed=b + k)
    x[1] = 0                                        # a zero row
    x[2] = gen.bf16_bits(torch.full((K,), 1.5, dtype=torch.bfloat16))     # all ties
    pos = oracle.calib_positions(b, k, _acts(32, K, seed=5)) if static else None
    enc = oracle.fp_encode(b, k, x, pos)
    e2, e4 = oracle.fp_tables()
    G = K // b
    a = bits_to_f32(x).astype(np.float64)
    dense_codes = _unpack4(enc.dq4)
    g2 = [Fraction(v) for v in E2M1_MAGS]
    g4 = [Fraction(float(v)) for v in e4[:0x7F]]
    for m in range(M):
        amax = np.abs(a[m]).max()
        idx = enc.idx[m] if enc.idx is not None else pos
        sel = (np.arange(G)[:, None] * b + idx.astype(np.int64)).ravel()
        assert len(set(sel.tolist())) == G * k and np.all(np.diff(idx.astype(int), axis=1) > 0)   # k per bank, ascending
        insel = np.zeros(K, bool)
        insel[sel] = True
        assert not dense_codes[m][insel].any()                           # supports disjoint
        if amax == 0:
            assert enc.s_hi[m] == 0 and enc.shift[m] == 0 and not enc.vals[m].any() and not enc.dq4[m].any()
            continue
        if not static:                                                   # brute-force selection
            for g in range(G):
                order = sorted(range(b), key=lambda j: (-abs(a[m, g * b + j]), j))[:k]
                assert sorted(order) == idx[g].tolist()
        inv = np.float32(256.0) / np.float32(amax)
        assert enc.s_hi[m] == np.float32(amax) / np.float32(256.0)
        rmax = np.abs(a[m][~insel]).max() if (~insel).any() else 0.0
        e = next(t for t in range(7) if Fraction(float(rmax)) * Fraction(float(inv)) / 2 ** t <= 6)
        assert enc.shift[m] == e and enc.s_lo[m] == enc.s_hi[m] * np.float32(2.0 ** e)
        for j in range(K):
            v = Fraction(float(a[m, j])) * Fraction(float(inv))
            if insel[j]:
                slot = int(np.where(sel == j)[0][0])
                code = int(enc.vals[m].ravel()[slot])
                want = _nearest_even(abs(v), g4)
                want = 0 if want == 0 else want | (0x80 if v < 0 else 0)
                assert code == want and enc.a8[m, j] == code
            else:
                v = v / 2 ** e
                want = _nearest_even(abs(v), g2)
                want = 0 if want == 0 else want | (8 if v < 0 else 0)
                assert int(dense_codes[m, j]) == want
                # the merged operand holds the dense value times 2^e exactly, and it is an E4M3 number
                assert e4[enc.a8[m, j]] == e2[want] * 2.0 ** e and abs(e4[enc.a8[m, j]]) <= 384
        # reconstruction: within half a grid step of each format
        xhat, _ = oracle.fp_decode(b, k, enc, pos)
        err = np.abs(xhat[m].astype(np.float64) - a[m])
        assert np.all(err[insel] <= np.abs(a[m][insel]) * 2.0 ** -4 + float(enc.s_hi[m]) * 2.0 ** -9)
        assert np.all(err[~insel] <= float(enc.s_lo[m]) * 1.0 + 1e-12)   # E2M1 spacing is at most 2 (half: 1)


def test_weights_against_exact_rationals():
    N, K = 12, 128
    W = gen.bf16_bits(gen.weights(N, K, seed=3))
    W[5] = 0
    pw = oracle.fp_pack_weights(W)
    e2, e4 = oracle.fp_tables()
    w = bits_to_f32(W).astype(np.float64)
    codes = _unpack4(pw.wq4)
    g2 = [Fraction(v) for v in E2M1_MAGS]
    for n in range(N):
        wmax = np.abs(w[n]).max()
        if wmax == 0:
            assert pw.s_w[n] == 0 and not codes[n].any()
            continue
        c = np.float32(6.0) / np.float32(wmax)
        assert pw.s_w[n] == np.float32(wmax) / np.float32(6.0)
        for j in range(K):
            v = Fraction(float(w[n, j])) * Fraction(float(c))
            want = _nearest_even(abs(v), g2)
            want = 0 if want == 0 else want | (8 if v < 0 else 0)
            assert int(codes[n, j]) == want
        assert np.abs(e2[codes[n]]).max() == 6.0
    assert np.array_equal(e4[pw.w8], e2[codes])                  # the 8-bit copy holds the same values


def test_gemm_is_the_fp64_product_of_the_dequantised_operands():
    b, k, M, N, K = 32, 4, 7, 9, 256
    x, W = _acts(M, K, seed=11), gen.bf16_bits(gen.weights(N, K, seed=11))
    enc, pw = oracle.fp_encode(b, k, x), oracle.fp_pack_weights(W)
    acc, sabs, ref32, out = oracle.fp_gemm(enc, pw)
    e2, e4 = oracle.fp_tables()
    av, wv = e4[enc.a8], e2[_unpack4(pw.wq4)]
    brute = np.array([[sum(Fraction(float(p)) * Fraction(float(q)) for p, q in zip(av[m], wv[n])) for n in range(N)] for m in range(M)])
    assert np.array_equal(acc, np.array([[np.float32(float(v)) for v in row] for row in brute]))
    assert np.allclose(sabs, np.abs(av) @ np.abs(wv).T, rtol=1e-6)
    assert np.array_equal(ref32, (acc * enc.s_hi[:, None]) * pw.s_w[None, :])
    # fp64 product of the decoded tensors: the merged operand times s_hi IS the decoded activation
    xhat, _ = oracle.fp_decode(b, k, enc)
    assert np.array_equal(xhat.astype(np.float64), av * enc.s_hi.astype(np.float64)[:, None])
    full = xhat.astype(np.float64) @ (wv * pw.s_w.astype(np.float64)[:, None]).T
    assert np.all(np.abs(ref32 - full) <= 4 * np.spacing(np.abs(full).astype(np.float32)) + 1e-30)
    # sampled form returns the same entries
    a2, _, r2, _ = oracle.fp_gemm(enc, pw, rows=[1, 5], cols=[0, 8, 3])
    assert np.array_equal(a2, acc[np.ix_([1, 5], [0, 8, 3])]) and np.array_equal(r2, ref32[np.ix_([1, 5], [0, 8, 3])])
