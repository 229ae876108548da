"""Parity of the floating-point variant (sparse FP8 E4M3 + dense FP4 E2M1 activations, FP4 weights)
with its CPU oracle, through the C ABI.

Codes, indices, scales, shifts and the merged 8-bit operand are bit-exact.  The GEMM accumulates
in fp32 on the tensor core in an order the hardware chooses, so its accumulators are compared
with the oracle's exactly summed ones within an accumulation-order bound, |gpu - exact| <=
2^-20 * sum_j |a_j w_j| (K <= 65536 additions of fp32 partial sums, each within 2^-24 relative of
values bounded by the sum of magnitudes, with a factor 16 of slack), and the bf16 outputs within
the path's 1e-2 relative tolerance plus that bound carried through the two scales."""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2512_05409_b200 as sq

pytestmark = pytest.mark.gpu
REL_TOL = 1e-2
ORDER_TOL = 2.0 ** -20


def _np(t):
    return t.detach().cpu().numpy()


def _setup(M, N, K, b, k, static, seed):
    fmt = sq.make_format(b, k, static)
    X = gen.activations(M, K, seed=seed, outlier_fraction=0.01, outlier_scale=20.0, device="cuda")
    W = gen.weights(N, K, seed=seed, device="cuda")
    pos = pos_ref = None
    if static:
        pos = sq.sq_calib_positions(fmt, gen.calibration_batch(64, K, seed=seed, device="cuda"), W)
        pos_ref = _np(pos)
    return fmt, X, W, pos, pos_ref


def _compare_encoded(enc, a8, ref):
    assert np.array_equal(_np(enc.dq4), ref.dq4)
    assert np.array_equal(_np(enc.vals).view(np.uint8), ref.vals)
    if ref.idx is not None:
        assert np.array_equal(_np(enc.idx), ref.idx)
    assert np.array_equal(_np(enc.shift), ref.shift)
    assert np.array_equal(_np(enc.s_hi).view(np.uint32), ref.s_hi.view(np.uint32))
    assert np.array_equal(_np(enc.s_lo).view(np.uint32), ref.s_lo.view(np.uint32))
    assert np.array_equal(_np(a8), ref.a8)


@pytest.mark.parametrize("b,k,static", [(64, 8, False), (64, 8, True), (128, 16, True), (32, 4, False), (128, 32, False),
                                        (64, 12, True), (32, 3, False)])
@pytest.mark.parametrize("M,N,K", [(200, 328, 384), (1, 8, 128), (130, 520, 1024)])
def test_fp_pipeline_small(b, k, static, M, N, K):
    fmt, X, W, pos, pos_ref = _setup(M, N, K, b, k, static, seed=M + b + k)
    w = sq.sq_fp_pack_weights(W)
    enc, a8 = sq.sq_fp_encode(fmt, X, pos)
    acc = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    out = sq.sq_fp_gemm(enc, a8, w, acc_out=acc)
    dec = sq.sq_fp_decode(fmt, enc, pos)
    assert sq.sq_device_status() == sq.SQ_OK
    w_ref = oracle.fp_pack_weights(gen.bf16_bits(W))
    enc_ref = oracle.fp_encode(b, k, gen.bf16_bits(X), pos_ref)
    assert np.array_equal(_np(w.wq4), w_ref.wq4) and np.array_equal(_np(w.w8), w_ref.w8)
    assert np.array_equal(_np(w.s_w).view(np.uint32), w_ref.s_w.view(np.uint32))
    _compare_encoded(enc, a8, enc_ref)
    assert np.array_equal(gen.bf16_bits(dec), oracle.fp_decode(b, k, enc_ref, pos_ref)[1])
    acc_ref, sabs, ref32, _ = oracle.fp_gemm(enc_ref, w_ref)
    assert np.all(np.abs(_np(acc).astype(np.float64) - acc_ref) <= ORDER_TOL * sabs.astype(np.float64))
    got = out.float().cpu().numpy().astype(np.float64)
    scale = np.abs(enc_ref.s_hi.astype(np.float64))[:, None] * np.abs(w_ref.s_w.astype(np.float64))[None, :]
    assert np.all(np.abs(got - ref32) <= REL_TOL * np.abs(ref32) + 2 * ORDER_TOL * sabs * scale)


def test_fp_degenerate_rows():
    K, b, k = 256, 64, 8
    X = gen.activations(6, K, seed=3, device="cpu").float()
    X[0] = 0
    X[1] = -3.0
    X[2] = 0
    X[2, 77] = 2.5
    X[3] = X[3].abs().clamp_min(0.5)
    X = X.to(torch.bfloat16).cuda()
    for static in (False, True):
        fmt = sq.make_format(b, k, static)
        pos = torch.arange(k, dtype=torch.uint8, device="cuda").repeat(K // b, 1).contiguous() if static else None
        enc, a8 = sq.sq_fp_encode(fmt, X, pos)
        _compare_encoded(enc, a8, oracle.fp_encode(b, k, gen.bf16_bits(X), None if pos is None else _np(pos)))
    assert sq.sq_device_status() == sq.SQ_OK


@pytest.mark.parametrize("K,b,k", [(2048, 64, 8), (3072, 32, 3), (7168, 128, 16), (8192, 64, 32), (28672, 128, 16)])
def test_fp_static_encode_staged_rows(K, b, k):
    """Static positions at row lengths the staged-row kernel takes (one, two and eight warps per row,
    half-word and byte masks), a ragged row count, and rows that are all zero, all equal, one-hot
    and dominated by an outlier (largest shift, saturating dense codes)."""
    M = 75
    fmt = sq.make_format(b, k, True)
    X = gen.activations(M, K, seed=K + k, outlier_fraction=0.01, outlier_scale=30.0, device="cpu").float()
    X[0] = 0
    X[1] = -3.0
    X[2] = 0
    X[2, K - 3] = 2.5
    X[3] = X[3].abs().clamp_min(0.5)
    X[4, 5] = 3.0e4
    X[M - 1] = 1.0
    X = X.to(torch.bfloat16).cuda()
    pos = sq.sq_calib_positions(fmt, gen.calibration_batch(64, K, seed=K, outlier_fraction=0.01, outlier_scale=30.0, device="cuda"))
    enc, a8 = sq.sq_fp_encode(fmt, X, pos)
    assert sq.sq_device_status() == sq.SQ_OK
    _compare_encoded(enc, a8, oracle.fp_encode(b, k, gen.bf16_bits(X), _np(pos)))


@pytest.mark.parametrize("static", [False, True])
def test_fp_dense_codes_at_every_input_near_the_grid(static):
    """The dense codes come from per-row thresholds on the bf16 input.  Every row here holds EVERY
    bf16 magnitude of the eleven binades below its maximum (both signs), so for each of 192 row
    scales every input next to every rounding boundary is present: a threshold off by one input,
    or a tie sent the wrong way, changes a code."""
    b, k, K, M = 64, 8, 4096, 192
    rng = np.random.default_rng(7)
    rows = np.zeros((M, K), dtype=np.uint16)
    for r in range(M):
        top = int(rng.integers(0x3000, 0x4F00))            # the row maximum's bf16 pattern (2^-31 .. 2^31)
        mags = np.arange(top - 11 * 128, top + 1, dtype=np.int64)   # eleven binades of consecutive patterns
        vals = np.concatenate([mags, mags | 0x8000]).astype(np.uint16)
        rng.shuffle(vals)
        row = np.resize(vals, K)
        row[int(rng.integers(0, K))] = top
        rows[r] = row
    X = torch.from_numpy(rows.view(np.int16)).view(torch.bfloat16).cuda()
    fmt = sq.make_format(b, k, static)
    pos = None
    if static:
        pos = torch.arange(k, dtype=torch.uint8, device="cuda").mul(7).remainder(b).sort().values.repeat(K // b, 1).contiguous()
    enc, a8 = sq.sq_fp_encode(fmt, X, pos)
    assert sq.sq_device_status() == sq.SQ_OK
    _compare_encoded(enc, a8, oracle.fp_encode(b, k, rows, None if pos is None else _np(pos)))


@pytest.mark.parametrize("static", [False, True])
def test_fp_full_size_sweep_shape(static):
    """M = 4096, K = N = 8192 (the format-sweep shape): every row's encoding in full, GEMM on sampled
    rows x channels."""
    M, N, K, b, k = 4096, 8192, 8192, 128, 16
    fmt, X, W, pos, pos_ref = _setup(M, N, K, b, k, static, seed=9)
    w = sq.sq_fp_pack_weights(W)
    enc, a8 = sq.sq_fp_encode(fmt, X, pos)
    acc = torch.empty(M, N, dtype=torch.float32, device="cuda")
    out = sq.sq_fp_gemm(enc, a8, w, acc_out=acc)
    out2 = sq.sq_fp_gemm(enc, a8, w)
    assert sq.sq_device_status() == sq.SQ_OK and torch.equal(out, out2)
    enc_ref = oracle.fp_encode(b, k, gen.bf16_bits(X), pos_ref)
    _compare_encoded(enc, a8, enc_ref)
    rng = np.random.default_rng(1)
    rows = np.unique(np.concatenate([[0, 127, 128, M - 1], rng.integers(0, M, 20)]))
    cols = np.unique(np.concatenate([[0, 255, 256, N - 1], rng.integers(0, N, 60)]))
    w_ref = oracle.fp_pack_weights(gen.bf16_bits(W)[cols])
    assert np.array_equal(_np(w.wq4)[cols], w_ref.wq4) and np.array_equal(_np(w.w8)[cols], w_ref.w8)
    acc_ref, sabs, ref32, _ = oracle.fp_gemm(enc_ref, w_ref, rows=rows)
    got_acc = _np(acc)[np.ix_(rows, cols)].astype(np.float64)
    assert np.all(np.abs(got_acc - acc_ref) <= ORDER_TOL * sabs)
    got = out.float().cpu().numpy()[np.ix_(rows, cols)].astype(np.float64)
    scale = np.abs(enc_ref.s_hi.astype(np.float64))[rows][:, None] * np.abs(w_ref.s_w.astype(np.float64))[None, :]
    assert np.all(np.abs(got - ref32) <= REL_TOL * np.abs(ref32) + 2 * ORDER_TOL * sabs * scale)
