"""Pins of the CPU oracle against what the paper and plain mathematics fix.

None of these tests touches the CUDA path.  Each pin is chosen so that a
plausible mistake in the oracle (a dropped term, a wrong sign or index, a
transposed operand, a wrong tie-break) makes it fail.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import gen
import oracle
from helpers import bits_to_f32, f32_to_bf16_bits, rne_fraction, sparse_dense_split, unpack_nibbles

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _acts(M, K, seed=0, **kw):
    return gen.bf16_bits(gen.activations(M, K, seed=seed, **kw))


def _wts(N, K, seed=0):
    return gen.bf16_bits(gen.weights(N, K, seed=seed))


# --------------------------------------------------------------------------- format accounting

def test_equivalent_bits_match_paper_table():
    """Section 4.1 notation + the printed y column of the appendix table."""
    n = 0
    with open(os.path.join(GOLDEN, "equivalent_bits.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            op, hh, hl, s, bits = line.split()
            got = oracle.equivalent_bits(float(hh), float(hl), float(s), on_weights=(op == "W"))
            assert got == float(bits), line
            n += 1
    assert n == 16


def test_two_four_sparsity_is_the_special_case():
    """Section 3.1: 2:4 sparsity is s=0.5, h_low=0, b=4: keep the 2 largest of every 4."""
    x = _acts(16, 64, seed=3, dist="normal", outlier_fraction=0.0)
    enc = oracle.encode(4, 2, x)
    mag = np.abs(bits_to_f32(x)).reshape(16, 16, 4)
    # textbook 2:4 magnitude pruning: the two largest of each group of four survive
    order = np.argsort(-mag, axis=-1, kind="stable")[..., :2]
    keep = np.sort(order, axis=-1)
    assert np.array_equal(enc.idx, keep.astype(np.uint8))
    assert oracle.equivalent_bits(8, 0, 0.5, on_weights=False) == 4.0


# --------------------------------------------------------------------------- dynamic selection

@pytest.mark.parametrize("b,k", [(32, 4), (64, 8), (64, 16), (128, 16), (64, 1), (16, 8)])
def test_dynamic_selection_is_topk_by_magnitude(b, k):
    M, K = 24, 4 * b
    x = _acts(M, K, seed=b + k)
    # force plenty of exact ties (bf16 has few mantissa bits, but make sure)
    x[:, ::7] = x[:, 3:4]
    enc = oracle.encode(b, k, x)
    mag = np.abs(bits_to_f32(x)).reshape(M, K // b, b)
    # brute force: full stable sort of each bank by (-mag, index)
    order = np.argsort(-mag, axis=-1, kind="stable")[..., :k]
    expect = np.sort(order, axis=-1).astype(np.uint8)
    assert np.array_equal(enc.idx, expect)
    # invariants: k per bank, < b, strictly ascending, selected >= unselected
    assert enc.idx.shape == (M, K // b, k) and enc.idx.max() < b
    assert np.all(np.diff(enc.idx.astype(int), axis=-1) > 0) or k == 1
    sel = np.zeros_like(mag, dtype=bool)
    np.put_along_axis(sel, enc.idx.astype(np.int64), True, axis=-1)
    lo_sel = np.where(sel, mag, np.inf).min(-1)
    hi_unsel = np.where(~sel, mag, -np.inf).max(-1)
    assert np.all(lo_sel >= hi_unsel)


def test_tie_break_prefers_lower_index():
    b, k = 32, 4
    x = np.full((1, b), 0x3F80, dtype=np.uint16)  # all 1.0
    enc = oracle.encode(b, k, x)
    assert enc.idx.ravel().tolist() == [0, 1, 2, 3]
    x[0, 10] = 0xC000  # -2.0 wins on magnitude, the other three are the first ties
    enc = oracle.encode(b, k, x)
    assert enc.idx.ravel().tolist() == [0, 1, 2, 10]


# --------------------------------------------------------------------------- encoding

def _exact_encode_row(a, sel_mask, kbits=None):
    """Exact-rational restatement of one row (Fractions; fp32 scale constants via numpy)."""
    amax = np.float32(np.max(np.abs(a)))
    if amax == 0:
        return np.zeros_like(a, dtype=np.int64), 0, np.float32(0)
    inv = np.float32(127.0) / amax
    rmax = np.float32(np.max(np.abs(a[~sel_mask]))) if (~sel_mask).any() else np.float32(0)
    e = 4
    for t in range(5):
        if rne_fraction(Fraction(float(rmax)) * Fraction(float(inv)) / (1 << t)) <= 7:
            e = t
            break
    q = np.zeros(a.shape, dtype=np.int64)
    for j, v in enumerate(a):
        if sel_mask[j]:
            q[j] = max(-127, min(127, rne_fraction(Fraction(float(v)) * Fraction(float(inv)))))
        else:
            q[j] = max(-7, min(7, rne_fraction(Fraction(float(v)) * Fraction(float(inv)) / (1 << e))))
    return q, e, inv


@pytest.mark.parametrize("mode", ["dynamic", "static"])
def test_encode_matches_exact_rational_arithmetic(mode):
    b, k, M, K = 32, 4, 6, 128
    x = _acts(M, K, seed=11)
    pos = None
    if mode == "static":
        pos = oracle.calib_positions(b, k, gen.bf16_bits(gen.calibration_batch(32, K, seed=11)))
    enc = oracle.encode(b, k, x, pos)
    q_lo, q_hi, sup = sparse_dense_split(enc, b, k, pos)
    a = bits_to_f32(x)
    for m in range(M):
        q, e, inv = _exact_encode_row(a[m], sup[m])
        assert enc.shift[m] == e
        assert np.array_equal(np.where(sup[m], q_hi[m], q_lo[m]), q)
        amax = np.float32(np.abs(a[m]).max())
        assert enc.s_hi[m] == amax / np.float32(127.0)
        assert enc.s_lo[m] == enc.s_hi[m] * np.float32(2.0 ** e)


@pytest.mark.parametrize("b,k,mode", [(64, 8, "dynamic"), (64, 8, "static"), (128, 16, "static"), (32, 2, "dynamic")])
def test_encoding_invariants_and_reconstruction(b, k, mode):
    M, K = 48, 1024
    x = _acts(M, K, seed=5)
    pos = None
    if mode == "static":
        pos = oracle.calib_positions(b, k, gen.bf16_bits(gen.calibration_batch(64, K, seed=5)))
    enc = oracle.encode(b, k, x, pos)
    q_lo, q_hi, sup = sparse_dense_split(enc, b, k, pos)
    # exactly k per bank; dense support disjoint from the sparse support; code ranges
    assert np.all(sup.reshape(M, K // b, b).sum(-1) == k)
    assert np.all(q_lo[sup] == 0)
    assert q_lo.min() >= -7 and q_lo.max() <= 7 and q_hi.min() >= -127 and q_hi.max() <= 127
    assert enc.shift.max() <= 4
    # reconstruction: within one quantisation step (half a step where nothing clamps)
    a = bits_to_f32(x).astype(np.float64)
    xhat, xhat_bits = oracle.decode(b, k, enc, pos)
    err = np.abs(a - xhat.astype(np.float64))
    s_hi = enc.s_hi.astype(np.float64)[:, None]
    s_lo = enc.s_lo.astype(np.float64)[:, None]
    slack = 1.0 + 2.0 ** -18
    assert np.all(err[sup] <= (np.broadcast_to(s_hi, err.shape)[sup] / 2) * slack + 1e-30)
    assert np.all(err[~sup] <= np.broadcast_to(s_lo, err.shape)[~sup] * slack + 1e-30)
    no_clamp = (enc.shift < 4)[:, None] & ~sup
    assert np.all(err[no_clamp] <= (np.broadcast_to(s_lo, err.shape)[no_clamp] / 2) * slack + 1e-30)
    assert np.array_equal(xhat_bits, f32_to_bf16_bits(xhat))


def _assert_equal_up_to_double_rounding(ours, textbook, prod32):
    """Equal, except where the textbook's fp32 product sits on (or an ulp from) a half-integer.

    The method rounds the exact product once.  A quantiser that first rounds the
    scale and the product to fp32 and then to an integer can differ by one only
    when that intermediate is a tie to within fp32 rounding.
    """
    diff = ours != textbook
    assert diff.mean() < 0.01
    assert np.all(np.abs(ours - textbook)[diff] == 1)
    p = np.abs(prod32[diff]).astype(np.float64)
    assert np.all(np.abs(p % 1.0 - 0.5) <= 4 * np.spacing(p.astype(np.float32)))


def test_shift_zero_rows_equal_textbook_per_token_int8():
    """With e = 0 the merged integer row is the per-token absmax INT8 quantisation of x."""
    b, k, M, K = 64, 8, 32, 256
    # mild rows: everything outside the top-k is below 7.5/127 of the row maximum
    base = bits_to_f32(_acts(M, K, seed=2, dist="normal", outlier_fraction=0.0))
    small = base * 0.01
    mag = np.abs(base).reshape(M, K // b, b)
    top = np.argsort(-mag, axis=-1, kind="stable")[..., :k]
    keep = np.zeros_like(mag, dtype=bool)
    np.put_along_axis(keep, top, True, axis=-1)
    x = np.where(keep.reshape(M, K), base, small).astype(np.float32)
    xb = f32_to_bf16_bits(x)
    enc = oracle.encode(b, k, xb)
    assert np.all(enc.shift == 0)
    q_lo, q_hi, sup = sparse_dense_split(enc, b, k)
    merged = q_lo + q_hi
    # textbook quantiser in torch fp32: round(x * 127 / amax)
    xt = torch.from_numpy(bits_to_f32(xb))
    amax = xt.abs().amax(dim=1, keepdim=True)
    prod32 = xt * (127.0 / amax)              # the textbook rounds this fp32 product a second time
    textbook = torch.round(prod32).clamp(-127, 127).to(torch.int64).numpy()
    _assert_equal_up_to_double_rounding(merged, textbook, prod32.numpy())
    # and k = b selects everything: the sparse component alone is that quantiser
    enc_all = oracle.encode(16, 16, xb)
    _assert_equal_up_to_double_rounding(enc_all.vals.reshape(M, K).astype(np.int64), textbook, prod32.numpy())
    assert np.all(enc_all.dq4 == 0)


def test_shift_thresholds():
    """e is the smallest shift for which the largest dense value fits in [-7, 7]."""
    b, k = 32, 1
    rows, expect = [], []
    # amax = 127 -> inv = 1: the dense maximum r needs e = min{e: rne(r / 2^e) <= 7}
    for r, e in [(7, 0), (7.5, 1), (8, 1), (14, 1), (15, 2), (15.5, 2), (29, 2), (30, 3), (31, 3),
                 (58, 3), (60, 4), (100, 4), (126, 4), (0, 0)]:
        row = np.zeros(b, dtype=np.float32)
        row[5] = 127.0
        row[9] = -r
        rows.append(row)
        expect.append(e)
    xb = f32_to_bf16_bits(np.stack(rows))
    enc = oracle.encode(b, k, xb)
    # ties go to even: 7.5 -> 8, 15/2 -> 8, 30/4 -> 8, 60/8 -> 8 all exceed 7 and need the next shift,
    # while 14/2, 29/4 = 7.25 and 58/8 = 7.25 still fit
    assert enc.shift.tolist() == expect
    q_lo, q_hi, sup = sparse_dense_split(enc, b, k)
    assert q_hi[:, 5].tolist() == [127] * len(rows)
    # value 126 at e = 4: 126/16 = 7.875 -> 8 -> clamped to 7 (sign kept)
    assert q_lo[12, 9] == -7


def test_degenerate_rows():
    b, k, K = 32, 4, 64
    zero = np.zeros((1, K), dtype=np.uint16)
    enc = oracle.encode(b, k, zero)
    assert enc.s_hi[0] == 0 and enc.s_lo[0] == 0 and enc.shift[0] == 0
    assert not enc.dq4.any() and not enc.vals.any()
    assert enc.idx.reshape(2, 4).tolist() == [[0, 1, 2, 3]] * 2
    const = f32_to_bf16_bits(np.full((1, K), -3.0, dtype=np.float32))
    enc = oracle.encode(b, k, const)
    q_lo, q_hi, sup = sparse_dense_split(enc, b, k)
    assert enc.shift[0] == 4 and np.all(q_hi[sup] == -127) and np.all(q_lo[~sup] == -7)
    one = np.zeros((1, K), dtype=np.float32)
    one[0, 40] = 2.5
    enc = oracle.encode(b, k, f32_to_bf16_bits(one))
    q_lo, q_hi, sup = sparse_dense_split(enc, b, k)
    assert enc.shift[0] == 0 and q_hi[0, 40] == 127 and q_hi.sum() == 127 and not q_lo.any()
    assert 8 in enc.idx[0, 1].tolist()


# --------------------------------------------------------------------------- static positions

def test_static_positions_rank_importance():
    b, k, T, K, N = 32, 4, 48, 256, 40
    calib = gen.bf16_bits(gen.calibration_batch(T, K, seed=9, outlier_fraction=0.02, outlier_scale=50.0))
    W = _wts(N, K, seed=9)
    pos, imp = oracle.calib_positions(b, k, calib, W, return_importance=True)
    # brute force in numpy: sequential fp64 sums (cumsum is sequential), then a stable ranking
    abar = np.cumsum(np.abs(bits_to_f32(calib).astype(np.float64)), axis=0)[-1] / T
    r = np.cumsum(bits_to_f32(W).astype(np.float64), axis=0)[-1]
    I = np.abs(abar * r)
    assert np.array_equal(imp, I)
    order = np.argsort(-I.reshape(K // b, b), axis=-1, kind="stable")[:, :k]
    assert np.array_equal(pos, np.sort(order, axis=-1).astype(np.uint8))
    # without weights the score is the mean magnitude alone
    pos0, imp0 = oracle.calib_positions(b, k, calib, None, return_importance=True)
    assert np.array_equal(imp0, abar)
    order0 = np.argsort(-abar.reshape(K // b, b), axis=-1, kind="stable")[:, :k]
    assert np.array_equal(pos0, np.sort(order0, axis=-1).astype(np.uint8))


def test_static_positions_pick_a_boosted_channel_and_use_the_weight_sum():
    b, k, T, K, N = 32, 2, 32, 64, 8
    rng = np.random.default_rng(0)
    calib = rng.standard_normal((T, K)).astype(np.float32)
    calib[:, 37] *= 50.0
    W = np.full((N, K), 0.02, dtype=np.float32)
    pos = oracle.calib_positions(b, k, f32_to_bf16_bits(calib), f32_to_bf16_bits(W))
    assert 37 - 32 in pos[1].tolist()
    # a channel whose weights cancel has zero importance no matter how large the activation
    W2 = W.copy()
    W2[: N // 2, 37] = -0.02
    pos2 = oracle.calib_positions(b, k, f32_to_bf16_bits(calib), f32_to_bf16_bits(W2))
    assert 37 - 32 not in pos2[1].tolist()
    # the sign of the sum does not matter (absolute value)
    pos3 = oracle.calib_positions(b, k, f32_to_bf16_bits(calib), f32_to_bf16_bits(-W))
    assert np.array_equal(pos3, pos)


# --------------------------------------------------------------------------- weights

def test_pack_weights_is_per_channel_absmax_int4():
    b, k, N, K = 32, 4, 12, 128
    W = _wts(N, K, seed=4)
    W[3] = 0  # a zero channel
    pos = oracle.calib_positions(b, k, gen.bf16_bits(gen.calibration_batch(16, K, seed=4)))
    pw = oracle.pack_weights(b, k, W, pos)
    w = bits_to_f32(W)
    for n in range(N):
        wmax = np.float32(np.abs(w[n]).max())
        if wmax == 0:
            assert pw.s_w[n] == 0 and not pw.wq[n].any()
            continue
        c = np.float32(7.0) / wmax
        exact = [max(-7, min(7, rne_fraction(Fraction(float(v)) * Fraction(float(c))))) for v in w[n]]
        assert pw.wq[n].tolist() == exact
        assert pw.s_w[n] == wmax / np.float32(7.0)
        assert np.abs(pw.wq[n]).max() == 7
    assert np.array_equal(unpack_nibbles(pw.wq4), pw.wq)
    assert np.array_equal(pw.colsum, pw.wq.astype(np.int64).sum(1).astype(np.int32))
    cols = (np.arange(K // b)[:, None] * b + pos.astype(np.int64)).ravel()
    assert np.array_equal(pw.w_sparse, pw.wq[:, cols])           # the gathered codes themselves
    # textbook torch quantiser agrees
    wt = torch.from_numpy(w)
    wm = wt.abs().amax(1, keepdim=True).clamp_min(1e-30)
    prod32 = wt * (7.0 / wm)
    tb = torch.round(prod32).clamp(-7, 7).to(torch.int64).numpy()
    _assert_equal_up_to_double_rounding(pw.wq.astype(np.int64), tb, prod32.numpy())


# --------------------------------------------------------------------------- GEMM

@pytest.mark.parametrize("b,k,mode", [(32, 4, "dynamic"), (64, 8, "static"), (64, 16, "dynamic")])
def test_integer_gemm_is_sum_of_component_gemms(b, k, mode):
    M, N, K = 20, 24, 256
    x, W = _acts(M, K, seed=21), _wts(N, K, seed=21)
    pos = None
    if mode == "static":
        pos = oracle.calib_positions(b, k, gen.bf16_bits(gen.calibration_batch(32, K, seed=21)), W)
    enc = oracle.encode(b, k, x, pos)
    pw = oracle.pack_weights(b, k, W, pos)
    acc, ref32, out = oracle.gemm(b, k, enc, pw, pos)
    q_lo, q_hi, sup = sparse_dense_split(enc, b, k, pos)
    wq = unpack_nibbles(pw.wq4).astype(np.int64)
    acc_lo = q_lo @ wq.T                      # dense INT4 x INT4 product
    acc_hi = q_hi @ wq.T                      # sparse INT8 x INT4 product
    expect = acc_lo * (1 << enc.shift.astype(np.int64))[:, None] + acc_hi
    assert np.array_equal(acc.astype(np.int64), expect)
    if mode == "static":                      # the sparse product through the reordered weights
        via_sparse = enc.vals.reshape(M, -1).astype(np.int64) @ pw.w_sparse.astype(np.int64).T
        assert np.array_equal(acc_hi, via_sparse)                # w_sparse holds the plain codes
    # epilogue definition and bf16 rounding
    ref = (acc.astype(np.float32) * enc.s_hi[:, None]) * pw.s_w[None, :]
    assert np.array_equal(ref, ref32)
    assert np.array_equal(out, f32_to_bf16_bits(ref32))
    # sampled form returns the same entries
    rows, cols = [3, 17, 0], [5, 23]
    a2, r2, o2 = oracle.gemm(b, k, enc, pw, pos, rows=rows, cols=cols)
    assert np.array_equal(a2, acc[np.ix_(rows, cols)]) and np.array_equal(r2, ref32[np.ix_(rows, cols)])


def test_gemm_matches_fp64_matmul_of_dequantised_operands():
    b, k, M, N, K = 32, 4, 9, 11, 128
    x, W = _acts(M, K, seed=33), _wts(N, K, seed=33)
    enc = oracle.encode(b, k, x)
    pw = oracle.pack_weights(b, k, W)
    acc, ref32, _ = oracle.gemm(b, k, enc, pw)
    q_lo, q_hi, sup = sparse_dense_split(enc, b, k)
    s_hi = enc.s_hi.astype(np.float64)[:, None]
    s_lo = enc.s_lo.astype(np.float64)[:, None]
    xhat = np.where(sup, s_hi * q_hi, s_lo * q_lo)                     # fp64, exact
    what = pw.s_w.astype(np.float64)[:, None] * unpack_nibbles(pw.wq4).astype(np.float64)
    brute = np.zeros((M, N))
    for m in range(M):
        for n in range(N):
            brute[m, n] = float(np.dot(xhat[m], what[n]))
    ulp = np.spacing(np.abs(ref32).astype(np.float32)).astype(np.float64)
    assert np.all(np.abs(ref32.astype(np.float64) - brute) <= 4 * ulp + 1e-300)
    # decode() is the same x^ (rounded once to fp32)
    xd, _ = oracle.decode(b, k, enc)
    assert np.array_equal(xd, xhat.astype(np.float32))


def test_shift_zero_gemm_equals_plain_w4a8():
    b, k, M, N, K = 64, 8, 8, 16, 256
    base = bits_to_f32(_acts(M, K, seed=2, dist="normal", outlier_fraction=0.0))
    mag = np.abs(base).reshape(M, K // b, b)
    top = np.argsort(-mag, axis=-1, kind="stable")[..., :k]
    keep = np.zeros_like(mag, dtype=bool)
    np.put_along_axis(keep, top, True, axis=-1)
    xb = f32_to_bf16_bits(np.where(keep.reshape(M, K), base, base * 0.01).astype(np.float32))
    W = _wts(N, K, seed=2)
    enc = oracle.encode(b, k, xb)
    assert np.all(enc.shift == 0)
    pw = oracle.pack_weights(b, k, W)
    acc, _, _ = oracle.gemm(b, k, enc, pw)
    xt = torch.from_numpy(bits_to_f32(xb))
    q_lo, q_hi, _ = sparse_dense_split(enc, b, k)
    prod32 = xt * (127.0 / xt.abs().amax(1, keepdim=True))
    a8 = torch.round(prod32).to(torch.int64).numpy()
    _assert_equal_up_to_double_rounding(q_lo + q_hi, a8, prod32.numpy())
    a8 = np.where(a8 != q_lo + q_hi, q_lo + q_hi, a8)   # take the single-rounding value at the ties
    assert np.array_equal(acc.astype(np.int64), a8 @ pw.wq.astype(np.int64).T)


# ----------------------------------------------------------------------------- independent scales (Algorithm 1's S_high / S_low)

def _indep_setup(b, k, M, N, K, seed):
    x, W = _acts(M, K, seed=seed), _wts(N, K, seed=seed)
    pos = oracle.calib_positions(b, k, gen.bf16_bits(gen.calibration_batch(32, K, seed=seed)), W)
    return x, W, pos


def test_indep_encode_matches_exact_rational_arithmetic():
    """Each part is a textbook symmetric quantiser with its own absmax scale: codes, scales and
    the half-step reconstruction bound, in exact rational arithmetic."""
    b, k, M, K = 32, 4, 6, 256
    x, _, pos = _indep_setup(b, k, M, 8, K, seed=41)
    enc = oracle.encode_indep(b, k, x, pos)
    assert enc.idx is None and np.all(enc.shift == 0)
    q_lo, q_hi, sup = sparse_dense_split(enc, b, k, pos)
    assert np.all(q_lo[sup] == 0) and np.all(q_hi[~sup] == 0)
    assert np.all(np.abs(q_lo) <= 7) and np.all(np.abs(q_hi) <= 127)
    a = bits_to_f32(x)
    for m in range(M):
        smax = np.float32(np.abs(a[m][sup[m]]).max())
        rmax = np.float32(np.abs(a[m][~sup[m]]).max())
        assert enc.s_hi[m] == smax / np.float32(127.0) and enc.s_lo[m] == rmax / np.float32(7.0)
        inv_hi, inv_lo = np.float32(127.0) / smax, np.float32(7.0) / rmax
        for j in range(K):
            inv, lim = (inv_hi, 127) if sup[m, j] else (inv_lo, 7)
            want = max(-lim, min(lim, rne_fraction(Fraction(float(a[m, j])) * Fraction(float(inv)))))
            assert (q_hi if sup[m, j] else q_lo)[m, j] == want
        # the extreme of each part takes the extreme code of its grid
        assert np.abs(q_hi[m]).max() == 127 and np.abs(q_lo[m]).max() == 7
    xd, _ = oracle.decode(b, k, enc, pos)
    step = np.where(sup, enc.s_hi[:, None], enc.s_lo[:, None]).astype(np.float64)
    assert np.all(np.abs(xd.astype(np.float64) - a) <= 0.5 * step * (1 + 1e-6) + 1e-30)


def test_indep_equals_tied_when_the_scales_are_a_power_of_two_apart():
    """Rows whose largest selected value is 127 * 2^p and whose largest other value is
    7 * 2^(p+e): both rules give the same inverse scales, so the same codes and, with the dense
    accumulator shifted by e, the same GEMM accumulator."""
    b, k, M, N, K = 32, 4, 5, 12, 128
    x, W, pos = _indep_setup(b, k, M, N, K, seed=43)
    a = bits_to_f32(x).copy()
    sup = np.zeros((M, K), dtype=bool)
    cols = (np.arange(K // b)[:, None] * b + pos.astype(np.int64)).reshape(-1)
    sup[:, cols] = True
    for m in range(M):
        e = m % 5
        a[m] = np.clip(a[m], -3.0, 3.0)
        a[m, cols[0]] = 127.0 * 0.125                      # the row maximum, at a selected place
        other = np.flatnonzero(~sup[m])
        a[m, other] = np.clip(a[m, other], -7.0 * 0.125 * 2 ** e, 7.0 * 0.125 * 2 ** e)
        a[m, other[m]] = -7.0 * 0.125 * 2 ** e             # the largest unselected magnitude
        sel = np.flatnonzero(sup[m])
        a[m, sel] = np.clip(a[m, sel], -127.0 * 0.125, 127.0 * 0.125)
    xb = f32_to_bf16_bits(a.astype(np.float32))
    tied = oracle.encode(b, k, xb, pos)
    ind = oracle.encode_indep(b, k, xb, pos)
    assert np.array_equal(tied.shift, np.arange(M) % 5)
    assert np.array_equal(tied.dq4, ind.dq4) and np.array_equal(tied.vals, ind.vals)
    assert np.array_equal(tied.s_hi, ind.s_hi) and np.array_equal(tied.s_lo, ind.s_lo)
    pw = oracle.pack_weights(b, k, W, pos)
    acc, ref32, out = oracle.gemm(b, k, tied, pw, pos)
    lo, hi, ref_i, out_i = oracle.gemm_indep(b, k, ind, pw, pos)
    assert np.array_equal((lo.astype(np.int64) << tied.shift[:, None].astype(np.int64)) + hi, acc.astype(np.int64))
    # the two epilogues round differently (one product of the merged sum against a fused
    # multiply-add of the two parts), but only in the last place
    ulp = np.spacing(np.abs(ref32))
    assert np.all(np.abs(ref_i - ref32) <= 2 * ulp)


def test_indep_gemm_is_two_integer_products_and_matches_fp64():
    b, k, M, N, K = 32, 8, 9, 11, 128
    x, W, pos = _indep_setup(b, k, M, N, K, seed=47)
    enc = oracle.encode_indep(b, k, x, pos)
    pw = oracle.pack_weights(b, k, W, pos)
    lo, hi, ref32, out = oracle.gemm_indep(b, k, enc, pw, pos)
    q_lo, q_hi, sup = sparse_dense_split(enc, b, k, pos)
    wq = pw.wq.astype(np.int64)
    assert np.array_equal(lo.astype(np.int64), q_lo @ wq.T)
    assert np.array_equal(hi.astype(np.int64), q_hi @ wq.T)
    # the gathered weight rows of Algorithm 2 give the same sparse product
    cols = (np.arange(K // b)[:, None] * b + pos.astype(np.int64)).reshape(-1)
    assert np.array_equal(hi.astype(np.int64), enc.vals.reshape(M, -1).astype(np.int64) @ pw.w_sparse.astype(np.int64).T)
    assert np.array_equal(pw.w_sparse.astype(np.int64), wq[:, cols])
    # fp64 brute force of the dequantised operands
    xhat = np.where(sup, enc.s_hi.astype(np.float64)[:, None] * q_hi, enc.s_lo.astype(np.float64)[:, None] * q_lo)
    what = pw.s_w.astype(np.float64)[:, None] * wq.astype(np.float64)
    brute = np.zeros((M, N))
    for m in range(M):
        for n in range(N):
            brute[m, n] = float(np.dot(xhat[m], what[n]))
    # fp32 epilogue: the two terms may cancel, so the bound is relative to their magnitudes
    scale = (np.abs(lo) * enc.s_lo[:, None] + np.abs(hi) * enc.s_hi[:, None]) * np.abs(pw.s_w)[None, :]
    assert np.all(np.abs(ref32.astype(np.float64) - brute) <= 4 * 2.0 ** -24 * scale + 1e-300)
    assert np.array_equal(out, f32_to_bf16_bits(ref32))
    # sampled form returns the same entries
    rows, cols2 = [3, 8, 0], [5, 10]
    lo2, hi2, r2, o2 = oracle.gemm_indep(b, k, enc, pw, pos, rows=rows, cols=cols2)
    assert np.array_equal(lo2, lo[np.ix_(rows, cols2)]) and np.array_equal(hi2, hi[np.ix_(rows, cols2)])
    assert np.array_equal(r2, ref32[np.ix_(rows, cols2)]) and np.array_equal(o2, out[np.ix_(rows, cols2)])


def test_indep_degenerate_rows():
    b, k, K = 32, 4, 64
    pos = np.tile(np.arange(k, dtype=np.uint8), (K // b, 1))
    a = np.zeros((3, K), dtype=np.float32)
    a[1, 0] = 5.0            # only a selected place is non-zero
    a[2, 10] = -3.0          # only an unselected place is non-zero
    enc = oracle.encode_indep(b, k, f32_to_bf16_bits(a), pos)
    assert np.array_equal(enc.s_hi, np.array([0, 5.0 / 127.0, 0], dtype=np.float32))
    assert np.array_equal(enc.s_lo, np.array([0, 0, 3.0 / 7.0], dtype=np.float32))
    q_lo, q_hi, _ = sparse_dense_split(enc, b, k, pos)
    assert not q_lo[0].any() and not q_hi[0].any()
    assert q_hi[1, 0] == 127 and not q_lo[1].any()
    assert q_lo[2, 10] == -7 and not q_hi[2].any()
