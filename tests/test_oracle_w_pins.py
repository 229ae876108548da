"""Pins of the weights-in-SQ-format oracle (format part of Algorithm 1): brute-force selection by
the given importance scores, exact rationals for every code, the implicit mask (the pattern 1000
exactly k times per bank and never as a value), the storage closed form of the paper's notation,
reconstruction bounds, and an fp64 brute-force product.  CPU only."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import gen
import oracle
from helpers import bits_to_f32, rne_fraction, unpack_nibbles


def _setup(N, K, seed):
    W = gen.bf16_bits(gen.weights(N, K, seed=seed))
    rng = np.random.default_rng(seed)
    imp = (bits_to_f32(W).astype(np.float64) ** 2 * rng.uniform(0.2, 5.0, (N, K))).astype(np.float32)
    return W, imp


@pytest.mark.parametrize("b,k", [(32, 4), (64, 8), (128, 32), (64, 5)])
def test_encode_selection_codes_and_mask(b, k):
    N, K = 10, 256
    W, imp = _setup(N, K, seed=b + k)
    imp[3, :] = 1.0                    # all ties in one channel: lower indices win
    W[4] = 0                           # an all-zero channel
    enc = oracle.w_encode(b, k, W, imp)
    w = bits_to_f32(W)
    G = K // b
    nib = (np.stack([enc.wq4 & 0xF, enc.wq4 >> 4], axis=-1).reshape(N, K)).astype(int)
    for n in range(N):
        sel = np.zeros(K, bool)
        for g in range(G):
            order = sorted(range(b), key=lambda j: (-float(imp[n, g * b + j]), j))[:k]
            sel[[g * b + j for j in order]] = True
            assert (nib[n, g * b:(g + 1) * b] == 8).sum() == k           # exactly k masked places per bank
        assert np.array_equal(nib[n] == 8, sel)                            # and they are the k most important
        hmax, lmax = np.abs(w[n][sel]).max(), np.abs(w[n][~sel]).max()
        if hmax == 0:
            assert enc.s_high[n] == 0 and not enc.w_hi[n].any()
        else:
            assert enc.s_high[n] == np.float32(hmax) / np.float32(127.0)
            inv = np.float32(127.0) / np.float32(hmax)
            want = [max(-127, min(127, rne_fraction(Fraction(float(v)) * Fraction(float(inv))))) for v in w[n][sel]]
            assert enc.w_hi[n].ravel().tolist() == want                    # compact, in position order
            assert np.abs(enc.w_hi[n]).max() == 127
        if lmax == 0:
            assert enc.s_low[n] == 0
        else:
            assert enc.s_low[n] == np.float32(lmax) / np.float32(7.0)
            inv = np.float32(7.0) / np.float32(lmax)
            want = [max(-7, min(7, rne_fraction(Fraction(float(v)) * Fraction(float(inv))))) & 0xF for v in w[n][~sel]]
            assert nib[n][~sel].tolist() == want                           # the mask pattern is never a value
    # storage: K/2 + (K/b)*k bytes per channel = ((1-s)*h_high + h_low)/8 bytes per element (Section 4.1)
    s = 1.0 - k / b
    assert (enc.wq4[0].nbytes + enc.w_hi[0].nbytes) * 8 / K == oracle.equivalent_bits(8, 4, s, True)
    # reconstruction within half a step of each part's grid (the scale and its reciprocal are rounded
    # separately, which can move a code's value by up to 127 * 2^-22 of a step)
    what = oracle.w_decode(b, k, enc)
    for n in range(N):
        sel = nib[n] == 8
        err = np.abs(what[n].astype(np.float64) - w[n])
        assert np.all(err[sel] <= enc.s_high[n] / 2 * (1 + 2.0 ** -12)) and np.all(err[~sel] <= enc.s_low[n] / 2 * (1 + 2.0 ** -12))


def test_activation_int8_is_the_textbook_per_token_quantiser():
    x = gen.bf16_bits(gen.activations(5, 384, seed=2, outlier_fraction=0.02, outlier_scale=20.0))
    x[3] = 0
    xq, s_x = oracle.act_quant8(x)
    a = bits_to_f32(x)
    for m in range(5):
        amax = np.abs(a[m]).max()
        if amax == 0:
            assert s_x[m] == 0 and not xq[m].any()
            continue
        inv = np.float32(127.0) / np.float32(amax)
        assert s_x[m] == np.float32(amax) / np.float32(127.0)
        assert xq[m].tolist() == [max(-127, min(127, rne_fraction(Fraction(float(v)) * Fraction(float(inv))))) for v in a[m]]
        assert np.abs(xq[m]).max() == 127


def test_gemm_is_two_integer_products_and_matches_fp64():
    b, k, M, N, K = 32, 4, 5, 12, 256
    W, imp = _setup(N, K, seed=9)
    enc = oracle.w_encode(b, k, W, imp)
    xq, s_x = oracle.act_quant8(gen.bf16_bits(gen.activations(M, K, seed=9)))
    lo, hi, ref32, out = oracle.w_gemm(b, k, xq, s_x, enc)
    nib = np.stack([enc.wq4 & 0xF, enc.wq4 >> 4], axis=-1).reshape(N, K).astype(np.int64)
    mask = nib == 8
    q_lo = np.where(mask, 0, np.where(nib >= 8, nib - 16, nib))
    q_hi = np.zeros((N, K), dtype=np.int64)
    q_hi[mask] = enc.w_hi.reshape(N, -1).ravel()          # row-major order of the mask = bank by bank, position order
    assert np.array_equal(lo.astype(np.int64), xq.astype(np.int64) @ q_lo.T)
    assert np.array_equal(hi.astype(np.int64), xq.astype(np.int64) @ q_hi.T)
    # epilogue: one fp32 product, one fused multiply-add (exact product + sum, rounded once), one product
    t = (lo.astype(np.float32) * enc.s_low[None, :]).astype(np.float64)
    fma = (hi.astype(np.float64) * enc.s_high.astype(np.float64)[None, :] + t).astype(np.float32)
    assert np.array_equal(ref32, fma * s_x[:, None])
    # fp64 brute force of the dequantised operands
    what = oracle.w_decode(b, k, enc).astype(np.float64)
    xhat = xq.astype(np.float64) * s_x.astype(np.float64)[:, None]
    full = xhat @ what.T
    assert np.all(np.abs(ref32 - full) <= 8 * np.spacing(np.abs(full).astype(np.float32)) + 1e-30)
    assert np.array_equal(out, (torch.from_numpy(ref32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)))
