"""Parity at the benchmark configurations' full sizes, in the launch configuration bench.py times.

Everything is row- (token-) or channel-independent, so the oracle recomputes SAMPLED token rows
and SAMPLED output channels from the same inputs and must agree bit for bit with what the full-size
launches produced at those places; static positions are compared in full.
"""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2512_05409_b200 as sq
from test_gpu_parity import assert_bf16_close, check_status, merged_operand_from_oracle, _np, _bits

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _sample(n, count, seed, always=()):
    rng = np.random.default_rng(seed)
    picks = np.concatenate([np.array(list(always), dtype=np.int64), rng.integers(0, n, count)])
    return np.unique(np.clip(picks, 0, n - 1))


class PackedLinear:
    """Weights of one linear packed on the GPU (and its oracle twin on sampled channels)."""

    def __init__(self, N, K, b, k, static, seed, calib_dist=None):
        self.N, self.K, self.b, self.k, self.static = N, K, b, k, static
        self.fmt = sq.make_format(b, k, static)
        self.W = gen.weights(N, K, seed=seed, device=DEV)
        self.pos = self.pos_ref = None
        if static:
            kw = calib_dist or {}
            calib = gen.calibration_batch(512, K, seed=seed, device=DEV, **kw)
            self.pos = sq.sq_calib_positions(self.fmt, calib, self.W)
            self.pos_ref = oracle.calib_positions(b, k, _bits(calib), _bits(self.W))
            assert np.array_equal(_np(self.pos), self.pos_ref)          # positions compared in full
        self.w = sq.sq_pack_weights(self.fmt, self.W, self.pos)
        self.cols = _sample(N, 48, seed + 1, always=(0, N - 1, min(255, N - 1), min(256, N - 1)))
        self.w_ref = oracle.pack_weights(b, k, _bits(self.W[torch.from_numpy(self.cols).to(DEV)]), self.pos_ref)
        assert np.array_equal(_np(self.w.wq4)[self.cols], self.w_ref.wq4)
        assert np.array_equal(_np(self.w.colsum)[self.cols], self.w_ref.colsum)
        assert np.array_equal(_np(self.w.s_w)[self.cols].view(np.uint32), self.w_ref.s_w.view(np.uint32))
        if static:
            assert np.array_equal(_np(self.w.w_sparse)[self.cols].astype(np.int16), 16 * self.w_ref.w_sparse.astype(np.int16))
        del self.W


def check_linear(lin: PackedLinear, X: torch.Tensor, seed: int, n_rows=24):
    """Encode + GEMM at full size on the GPU; oracle on sampled rows x sampled channels."""
    M = X.shape[0]
    enc = sq.sq_encode(lin.fmt, X, lin.pos)
    acc = torch.empty(M, lin.N, dtype=torch.int32, device=DEV)
    out = sq.sq_gemm(lin.fmt, enc, lin.w, lin.pos, acc_out=acc)
    check_status()
    rows = _sample(M, n_rows, seed, always=(0, M - 1, min(127, M - 1), min(128, M - 1), min(255, M - 1), min(256, M - 1)))
    rows_t = torch.from_numpy(rows).to(DEV)
    enc_ref = oracle.encode(lin.b, lin.k, _bits(X[rows_t]), lin.pos_ref)
    assert np.array_equal(_np(enc.dq4[rows_t]), enc_ref.dq4)
    assert np.array_equal(_np(enc.vals[rows_t]), enc_ref.vals)
    if not lin.static:
        assert np.array_equal(_np(enc.idx[rows_t]), enc_ref.idx)
    assert np.array_equal(_np(enc.shift[rows_t]), enc_ref.shift)
    assert np.array_equal(_np(enc.s_hi[rows_t]).view(np.uint32), enc_ref.s_hi.view(np.uint32))
    assert np.array_equal(_np(enc.s_lo[rows_t]).view(np.uint32), enc_ref.s_lo.view(np.uint32))
    acc_ref, ref32, out_ref = oracle.gemm(lin.b, lin.k, enc_ref, lin.w_ref, lin.pos_ref)
    cols_t = torch.from_numpy(lin.cols).to(DEV)
    assert np.array_equal(_np(acc[rows_t][:, cols_t]), acc_ref)
    assert_bf16_close(out[rows_t][:, cols_t], ref32)
    # the binding's sq_gemm hands the library a workspace (split-K for few rows, pre-widened activations
    # for dynamic positions); the plain call must give the same bits
    plain = sq.sq_gemm(lin.fmt, enc, lin.w, lin.pos, use_workspace=False)
    check_status()
    assert torch.equal(plain, out)
    del plain
    # the pair bench.py's step calls: the encode that also writes the product's merged 8-bit operand,
    # and the product that reads it
    enc2, a8 = sq.sq_encode_a8(lin.fmt, X, lin.pos)
    check_status()
    for got, want in ((enc2.dq4, enc.dq4), (enc2.vals, enc.vals), (enc2.shift, enc.shift)):
        assert torch.equal(got, want)
    assert torch.equal(enc2.s_hi.view(torch.int32), enc.s_hi.view(torch.int32))
    assert torch.equal(enc2.s_lo.view(torch.int32), enc.s_lo.view(torch.int32))
    if not lin.static:
        assert torch.equal(enc2.idx, enc.idx)
    assert np.array_equal(_np(a8[rows_t]), merged_operand_from_oracle(lin.b, lin.k, enc_ref, lin.pos_ref))
    acc2 = torch.empty(M, lin.N, dtype=torch.int32, device=DEV)
    out2 = sq.sq_gemm_a8(lin.fmt, enc2, a8, lin.w, lin.pos, acc_out=acc2)
    check_status()
    assert np.array_equal(_np(acc2[rows_t][:, cols_t]), acc_ref)
    assert torch.equal(out2, out)
    del acc, out, enc, enc2, a8, acc2, out2


# ----------------------------------------------------------------------------- config 2: sq_encode alone

@pytest.mark.parametrize("static", [False, True])
@pytest.mark.parametrize("k", [4, 8, 16])
def test_config2_encode_8192x8192_in_full(k, static):
    M = K = 8192
    b = 64
    fmt = sq.make_format(b, k, static)
    X = gen.activations(M, K, seed=0, outlier_fraction=0.005, outlier_scale=50.0, device=DEV)
    pos = pos_ref = None
    if static:
        calib = gen.calibration_batch(512, K, seed=0, outlier_fraction=0.005, outlier_scale=50.0, device=DEV)
        pos = sq.sq_calib_positions(fmt, calib)
        pos_ref = oracle.calib_positions(b, k, _bits(calib))
        assert np.array_equal(_np(pos), pos_ref)
    enc = sq.sq_encode(fmt, X, pos)
    check_status()
    ref = oracle.encode(b, k, _bits(X), pos_ref)       # every row, every element
    assert np.array_equal(_np(enc.dq4), ref.dq4)
    assert np.array_equal(_np(enc.vals), ref.vals)
    if not static:
        assert np.array_equal(_np(enc.idx), ref.idx)
    assert np.array_equal(_np(enc.shift), ref.shift)
    assert np.array_equal(_np(enc.s_hi).view(np.uint32), ref.s_hi.view(np.uint32))
    assert np.array_equal(_np(enc.s_lo).view(np.uint32), ref.s_lo.view(np.uint32))
    rows = _sample(M, 16, k, always=(0, M - 1))
    dec = sq.sq_decode(fmt, enc, pos)
    sub = oracle.Encoded(ref.dq4[rows], ref.vals[rows], None if static else ref.idx[rows], ref.s_hi[rows],
                         ref.s_lo[rows], ref.shift[rows])
    assert np.array_equal(_bits(dec[torch.from_numpy(rows).to(DEV)]), oracle.decode(b, k, sub, pos_ref)[1])


# ----------------------------------------------------------------------------- config 3: 8B-shaped linears

@pytest.mark.parametrize("K,N", [(4096, 6144), (4096, 4096), (4096, 28672), (14336, 4096)])
def test_config3_8b_linears_dynamic(K, N):
    lin = PackedLinear(N, K, 64, 8, False, seed=K + N)
    for M in (1, 16, 128, 2048):
        X = gen.activations(M, K, seed=M, outlier_fraction=0.01, outlier_scale=20.0, device=DEV)
        check_linear(lin, X, seed=M)


# ----------------------------------------------------------------------------- config 4: 70B-shaped prefill

@pytest.mark.parametrize("K,N", [(8192, 10240), (8192, 8192), (8192, 57344), (28672, 8192)])
def test_config4_70b_prefill_static(K, N):
    lin = PackedLinear(N, K, 128, 16, True, seed=K + N,
                       calib_dist=dict(outlier_fraction=0.01, outlier_scale=20.0))
    X = gen.activations(4096, K, seed=K + N, outlier_fraction=0.01, outlier_scale=20.0, device=DEV)
    check_linear(lin, X, seed=7)


# ----------------------------------------------------------------------------- config 5: format sweep

@pytest.mark.parametrize("static", [False, True])
@pytest.mark.parametrize("b", [32, 64, 128])
def test_config5_format_sweep(b, static):
    M, K, N = 4096, 8192, 8192
    for frac_den in (16, 8, 4):
        k = b // frac_den
        for scale in (10.0, 50.0):
            lin = PackedLinear(N, K, b, k, static, seed=b + k,
                               calib_dist=dict(outlier_fraction=0.01, outlier_scale=scale))
            X = gen.activations(M, K, seed=int(scale), outlier_fraction=0.01, outlier_scale=scale, device=DEV)
            check_linear(lin, X, seed=k, n_rows=12)
            del lin, X
            torch.cuda.empty_cache()


# ----------------------------------------------------------------------------- independent scales at full size

@pytest.mark.parametrize("K,N,b,k", [(8192, 8192, 128, 16), (28672, 8192, 128, 16), (8192, 8192, 64, 8)])
def test_independent_scales_full_size(K, N, b, k):
    """SQ_POS_STATIC_INDEP at M = 4096: sampled rows x sampled channels of both accumulators and
    of the output against the oracle."""
    M = 4096
    lin = PackedLinear(N, K, b, k, True, seed=K + N + 1, calib_dist=dict(outlier_fraction=0.01, outlier_scale=20.0))
    fmt = sq.make_format(b, k, True, independent_scales=True)
    X = gen.activations(M, K, seed=K + N + 1, outlier_fraction=0.01, outlier_scale=20.0, device=DEV)
    enc = sq.sq_encode(fmt, X, lin.pos)
    acc = torch.empty(2, M, N, dtype=torch.int32, device=DEV)
    out = sq.sq_gemm(fmt, enc, lin.w, lin.pos, acc_out=acc)
    check_status()
    rows = _sample(M, 16, 3, always=(0, M - 1, 127, 128, 255, 256))
    rows_t, cols_t = torch.from_numpy(rows).to(DEV), torch.from_numpy(lin.cols).to(DEV)
    enc_ref = oracle.encode_indep(b, k, _bits(X[rows_t]), lin.pos_ref)
    assert np.array_equal(_np(enc.dq4[rows_t]), enc_ref.dq4) and np.array_equal(_np(enc.vals[rows_t]), enc_ref.vals)
    assert np.array_equal(_np(enc.s_hi[rows_t]).view(np.uint32), enc_ref.s_hi.view(np.uint32))
    assert np.array_equal(_np(enc.s_lo[rows_t]).view(np.uint32), enc_ref.s_lo.view(np.uint32))
    assert not _np(enc.shift[rows_t]).any()
    lo, hi, ref32, out_ref = oracle.gemm_indep(b, k, enc_ref, lin.w_ref, lin.pos_ref)
    assert np.array_equal(_np(acc[0][rows_t][:, cols_t]), lo) and np.array_equal(_np(acc[1][rows_t][:, cols_t]), hi)
    assert_bf16_close(out[rows_t][:, cols_t], ref32)
    assert np.array_equal(_bits(out[rows_t][:, cols_t].contiguous()), out_ref)
