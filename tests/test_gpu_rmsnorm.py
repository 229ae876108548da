"""The normalisation fused into the static-position encode (sq_rmsnorm_encode) against the oracle:
every integer, both scales and the merged 8-bit operand bit for bit; what it does not take is
refused before anything is launched."""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2512_05409_b200 as sq
from test_gpu_parity import _bits, _np, check_status, compare_encoded, merged_operand_from_oracle

pytestmark = pytest.mark.gpu


def _gamma(K, seed, device="cuda"):
    return (1.0 + 0.25 * gen.weights(1, K, seed=seed, std=1.0, device=device).float()).to(torch.bfloat16).reshape(K).contiguous()


@pytest.mark.parametrize("want_a8", [False, True])
@pytest.mark.parametrize("M,K,b,k", [
    (300, 2048, 64, 8),       # one warp per row
    (1, 2048, 64, 8),
    (130, 3072, 32, 4),
    (1500, 4096, 128, 16),    # more rows than row groups in flight: the slots are refilled
    (700, 8192, 64, 8),       # two warps per row: the mean of squares crosses warps
    (257, 8192, 128, 32),
    (90, 7168, 128, 16),
])
def test_rmsnorm_encode_matches_the_oracle(M, K, b, k, want_a8):
    fmt = sq.make_format(b, k, True)
    X = gen.activations(M, K, seed=M + K, outlier_fraction=0.01, outlier_scale=30.0, device="cuda")
    gamma = _gamma(K, seed=K + b)
    eps = 1e-5
    pos = sq.sq_calib_positions(fmt, gen.calibration_batch(64, K, seed=K, outlier_fraction=0.01, outlier_scale=30.0, device="cuda"), None)
    keep = X.clone()
    a8 = torch.full((M, K), 0x5A, dtype=torch.uint8, device="cuda") if want_a8 else None
    enc, a8 = sq.sq_rmsnorm_encode(fmt, X, gamma, eps, pos, a8=a8, want_a8=want_a8)
    check_status()
    assert torch.equal(X, keep)
    pos_ref = _np(pos)
    enc_ref, y = oracle.rmsnorm_encode(b, k, _bits(X), _bits(gamma), eps, pos_ref)
    compare_encoded(enc, enc_ref)
    if want_a8:
        assert np.array_equal(_np(a8), merged_operand_from_oracle(b, k, enc_ref, pos_ref))
        # ... which is what the unfused pair of calls writes for the normalised rows
        y_t = torch.from_numpy(y.view(np.int16)).cuda().view(torch.bfloat16)
        enc2, a8_2 = sq.sq_encode_a8(fmt, y_t, pos)
        assert torch.equal(a8, a8_2) and torch.equal(enc.dq4, enc2.dq4) and torch.equal(enc.vals, enc2.vals)


def test_rmsnorm_encode_degenerate_rows():
    """Zero rows (r = 1/sqrt(eps), all codes zero), constant rows, one huge value, tiny rows."""
    M, K, b, k = 8, 4096, 64, 8
    fmt = sq.make_format(b, k, True)
    X = gen.activations(M, K, seed=3, device="cuda")
    X[0] = 0
    X[1] = 0.75
    X[2] = 0
    X[2, 1234] = 3.0e4
    X[3] *= 2.0 ** -60
    X[4] *= 2.0 ** 50
    X[5, ::2] = 0
    gamma = _gamma(K, seed=9)
    pos = sq.sq_calib_positions(fmt, gen.calibration_batch(64, K, seed=3, device="cuda"), None)
    for eps in (1e-6, 0.0):
        Xe = X.clone()
        if eps == 0.0:
            Xe[0] = 1.0      # a zero row without eps has no defined reciprocal root
        enc, a8 = sq.sq_rmsnorm_encode(fmt, Xe, gamma, eps, pos)
        check_status()
        enc_ref, _ = oracle.rmsnorm_encode(b, k, _bits(Xe), _bits(gamma), eps, _np(pos))
        compare_encoded(enc, enc_ref)
        assert np.array_equal(_np(a8), merged_operand_from_oracle(b, k, enc_ref, _np(pos)))


def test_rmsnorm_encode_refuses_what_it_does_not_take():
    X = gen.activations(16, 1024, seed=1, device="cuda")
    gamma = _gamma(1024, seed=2)
    pos = sq.sq_calib_positions(sq.make_format(64, 8, True), gen.calibration_batch(64, 1024, seed=1, device="cuda"), None)
    with pytest.raises(sq.SqError) as e:       # a row length its kernel does not take
        sq.sq_rmsnorm_encode(sq.make_format(64, 8, True), X, gamma, 1e-5, pos)
    assert e.value.status == sq.SQ_ERR_UNSUPPORTED
    X2 = gen.activations(16, 2048, seed=1, device="cuda")
    g2 = _gamma(2048, seed=2)
    with pytest.raises(sq.SqError) as e:       # dynamic positions at a ratio k/b the row-group kernel does not take
        sq.sq_rmsnorm_encode(sq.make_format(64, 5, False), X2, g2, 1e-5, None)
    assert e.value.status == sq.SQ_ERR_UNSUPPORTED
    pos2 = sq.sq_calib_positions(sq.make_format(64, 8, True), gen.calibration_batch(64, 2048, seed=1, device="cuda"), None)
    with pytest.raises(sq.SqError) as e:       # independent scales
        sq.sq_rmsnorm_encode(sq.make_format(64, 8, True, independent_scales=True), X2, g2, 1e-5, pos2)
    assert e.value.status == sq.SQ_ERR_UNSUPPORTED
    with pytest.raises(sq.SqError) as e:
        sq.sq_rmsnorm_encode(sq.make_format(64, 8, True), X2, g2, -1.0, pos2)
    assert e.value.status == sq.SQ_ERR_INVALID_ARG
    check_status()


@pytest.mark.parametrize("M,K,b,k", [(4096, 8192, 128, 16), (2048, 4096, 64, 8), (8192, 8192, 64, 8)])
def test_rmsnorm_encode_at_the_benchmark_sizes(M, K, b, k):
    """The launch configurations bench.py times (the inputs of the 70B- and 8B-shaped QKV and gate-up
    projections, and the 8192 x 8192 bandwidth test): sampled rows against the oracle, every row
    for sane scales."""
    fmt = sq.make_format(b, k, True)
    X = gen.activations(M, K, seed=M + K + 1, dist="student_t3", outlier_fraction=0.005, outlier_scale=50.0, device="cuda")
    gamma = _gamma(K, seed=K + 3)
    pos = sq.sq_calib_positions(fmt, gen.calibration_batch(512, K, seed=K + 1, dist="student_t3", outlier_fraction=0.005, outlier_scale=50.0, device="cuda"), None)
    enc, a8 = sq.sq_rmsnorm_encode(fmt, X, gamma, 1e-5, pos)
    check_status()
    rng = np.random.default_rng(M + K)
    rows = np.unique(np.concatenate([[0, 1, 147, 148, 1183, 1184, M - 1], rng.integers(0, M, size=40)]))
    rows_t = torch.from_numpy(rows).cuda()
    pos_ref = _np(pos)
    enc_ref, y = oracle.rmsnorm_encode(b, k, _bits(X[rows_t]), _bits(gamma), 1e-5, pos_ref)
    assert np.array_equal(_np(enc.dq4[rows_t]), enc_ref.dq4) and np.array_equal(_np(enc.vals[rows_t]), enc_ref.vals)
    assert np.array_equal(_np(enc.shift[rows_t]), enc_ref.shift)
    assert np.array_equal(_np(enc.s_hi[rows_t]).view(np.uint32), enc_ref.s_hi.view(np.uint32))
    assert np.array_equal(_np(enc.s_lo[rows_t]).view(np.uint32), enc_ref.s_lo.view(np.uint32))
    assert np.array_equal(_np(a8[rows_t]), merged_operand_from_oracle(b, k, enc_ref, pos_ref))
    # every row: scales are positive and finite, the largest INT8 magnitude of a row is 127
    assert torch.isfinite(enc.s_hi).all() and (enc.s_hi > 0).all()
    assert int(enc.vals.view(M, -1).abs().max(dim=1).values.min()) <= 127


@pytest.mark.parametrize("M,K,b,k", [(75, 2048, 64, 8), (300, 4096, 128, 16), (513, 8192, 64, 8), (40, 7168, 128, 32)])
def test_fp_rmsnorm_encode_matches_the_oracle(M, K, b, k):
    """The floating-point variant's encode of the normalised rows, the normalisation inside the kernel:
    codes, scales and the merged E4M3 operand against the oracle's encode of the oracle's normalisation."""
    from test_gpu_fp_variant import _compare_encoded
    fmt = sq.make_format(b, k, True)
    X = gen.activations(M, K, seed=M + K + 2, outlier_fraction=0.01, outlier_scale=30.0, device="cuda")
    X[0] = 0
    X[1] = -3.0
    gamma = _gamma(K, seed=K + 5)
    pos = sq.sq_calib_positions(fmt, gen.calibration_batch(64, K, seed=K, outlier_fraction=0.01, outlier_scale=30.0, device="cuda"), None)
    enc, a8 = sq.sq_fp_rmsnorm_encode(fmt, X, gamma, 1e-5, pos)
    check_status()
    y, _, ambiguous = oracle.rmsnorm(_bits(X), _bits(gamma), 1e-5)
    assert not ambiguous.any()
    _compare_encoded(enc, a8, oracle.fp_encode(b, k, y, _np(pos)))
    with pytest.raises(sq.SqError) as e:
        sq.sq_fp_rmsnorm_encode(sq.make_format(b, k, False), X, gamma, 1e-5, None)
    assert e.value.status == sq.SQ_ERR_UNSUPPORTED


@pytest.mark.parametrize("want_a8", [False, True])
@pytest.mark.parametrize("M,K,b,k", [
    (1, 4096, 64, 8),         # decode: one token
    (16, 4096, 64, 8),
    (16, 14336, 64, 8),       # the down projection's row length
    (300, 2048, 32, 4),
    (200, 4096, 128, 16),
    (700, 8192, 64, 16),
    (150, 1024, 64, 32),
])
def test_rmsnorm_encode_dynamic_positions(M, K, b, k, want_a8):
    """Dynamic positions (the k largest magnitudes of every bank of the NORMALISED row): the row is
    normalised in shared memory before the selection; codes, indices, scales and (expanded from
    them) the merged operand against the oracle."""
    fmt = sq.make_format(b, k, False)
    X = gen.activations(M, K, seed=M + K + 7, outlier_fraction=0.01, outlier_scale=30.0, device="cuda")
    if M > 2:
        X[1] = 0
        X[2] = 0.75
    gamma = _gamma(K, seed=K + b + 1)
    eps = 1e-5
    keep = X.clone()
    a8 = torch.full((M, K), 0x5A, dtype=torch.uint8, device="cuda") if want_a8 else None
    enc, a8 = sq.sq_rmsnorm_encode(fmt, X, gamma, eps, None, a8=a8, want_a8=want_a8)
    check_status()
    assert torch.equal(X, keep)
    enc_ref, _ = oracle.rmsnorm_encode(b, k, _bits(X), _bits(gamma), eps, None)
    compare_encoded(enc, enc_ref)
    if want_a8:
        assert np.array_equal(_np(a8), merged_operand_from_oracle(b, k, enc_ref, None))


def test_rmsnorm_encode_then_few_token_product_in_a_chain():
    """The decode chain normalisation+encode -> product, back to back over changing tokens, against
    the oracle's product of the oracle's encoding."""
    fmt = sq.make_format(64, 8, False)
    M, K, N = 16, 4096, 520
    W = gen.weights(N, K, seed=31, device="cuda")
    w = sq.sq_pack_weights(fmt, W)
    w_ref = oracle.pack_weights(64, 8, _bits(W))
    gamma = _gamma(K, seed=32)
    Xs = [gen.activations(M, K, seed=200 + i, outlier_fraction=0.01, outlier_scale=20.0, device="cuda") for i in range(4)]
    enc = sq.alloc_encoded(fmt, M, K, "cuda")
    outs = [torch.empty(M, N, dtype=torch.bfloat16, device="cuda") for _ in Xs]
    for X, out in zip(Xs, outs):
        sq.sq_rmsnorm_encode(fmt, X, gamma, 1e-5, None, out=enc, want_a8=False)
        sq.sq_gemm(fmt, enc, w, out=out)
    torch.cuda.synchronize()
    check_status()
    for X, out in zip(Xs, outs):
        enc_ref, _ = oracle.rmsnorm_encode(64, 8, _bits(X), _bits(gamma), 1e-5, None)
        _, _, out_ref = oracle.gemm(64, 8, enc_ref, w_ref)
        assert np.array_equal(_bits(out), out_ref)
