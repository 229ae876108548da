"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same seeded inputs.

Integers (packed nibbles, INT8 values, indices, shifts, positions, accumulators) must be
bit-exact; scales are produced by the same IEEE operations and must be bit-exact too; bf16
outputs must be within a relative error of 1e-2 of the oracle's fp32 result (they are in
fact equal unless a rounding mode differs).
"""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2512_05409_b200 as sq
from helpers import bits_to_f32

pytestmark = pytest.mark.gpu

REL_TOL = 1e-2   # max |gpu - ref32| / |ref32| for bf16 outputs (exact zero where ref32 == 0)


def _np(t):
    return t.detach().cpu().numpy()


def _bits(t):
    return gen.bf16_bits(t)


def assert_bf16_close(gpu_bf16: torch.Tensor, ref32: np.ndarray):
    got = gpu_bf16.float().cpu().numpy().astype(np.float64)
    ref = ref32.astype(np.float64)
    zero = ref == 0
    assert np.all(got[zero] == 0)
    rel = np.abs(got[~zero] - ref[~zero]) / np.abs(ref[~zero])
    assert rel.size == 0 or rel.max() <= REL_TOL, rel.max()


def check_status():
    assert sq.sq_device_status() == sq.SQ_OK


def compare_encoded(enc_gpu: sq.Encoded, enc_ref: oracle.Encoded, rows=None):
    sl = slice(None) if rows is None else rows
    assert np.array_equal(_np(enc_gpu.dq4)[sl], enc_ref.dq4)
    assert np.array_equal(_np(enc_gpu.vals)[sl], enc_ref.vals)
    if enc_ref.idx is not None:
        assert np.array_equal(_np(enc_gpu.idx)[sl], enc_ref.idx)
    assert np.array_equal(_np(enc_gpu.shift)[sl], enc_ref.shift)
    assert np.array_equal(_np(enc_gpu.s_hi)[sl].view(np.uint32), enc_ref.s_hi.view(np.uint32))
    assert np.array_equal(_np(enc_gpu.s_lo)[sl].view(np.uint32), enc_ref.s_lo.view(np.uint32))


def compare_weights(w_gpu: sq.Weights, w_ref: oracle.Weights, rows=None):
    sl = slice(None) if rows is None else rows
    assert np.array_equal(_np(w_gpu.wq4)[sl], w_ref.wq4)
    assert np.array_equal(_np(w_gpu.colsum)[sl], w_ref.colsum)
    assert np.array_equal(_np(w_gpu.s_w)[sl].view(np.uint32), w_ref.s_w.view(np.uint32))
    if w_ref.w_sparse is not None:
        # library layout: the gathered codes are stored in sixteenths (the unit of the GEMM's INT8
        # weight operand); the oracle holds the codes themselves
        assert np.array_equal(_np(w_gpu.w_sparse)[sl].astype(np.int16), 16 * w_ref.w_sparse.astype(np.int16))


def run_pipeline(M, N, K, b, k, static, seed=0, dist="student_t3", frac=0.01, scale=20.0, T=64,
                 X=None, full_gemm=True):
    """Whole path on the GPU vs the oracle; returns nothing, asserts everything."""
    dev = "cuda"
    fmt = sq.make_format(b, k, static)
    if X is None:
        X = gen.activations(M, K, seed=seed, dist=dist, outlier_fraction=frac, outlier_scale=scale, device=dev)
    W = gen.weights(N, K, seed=seed, device=dev)
    Xb, Wb = _bits(X), _bits(W)

    pos = pos_ref = None
    if static:
        calib = gen.calibration_batch(T, K, seed=seed, dist=dist, outlier_fraction=frac, outlier_scale=scale,
                                      device=dev)
        pos = sq.sq_calib_positions(fmt, calib, W)
        pos_ref = oracle.calib_positions(b, k, _bits(calib), Wb)
        assert np.array_equal(_np(pos), pos_ref)

    w_gpu = sq.sq_pack_weights(fmt, W, pos)
    w_ref = oracle.pack_weights(b, k, Wb, pos_ref)
    compare_weights(w_gpu, w_ref)

    enc_gpu = sq.sq_encode(fmt, X, pos)
    enc_ref = oracle.encode(b, k, Xb, pos_ref)
    compare_encoded(enc_gpu, enc_ref)

    dec_gpu = sq.sq_decode(fmt, enc_gpu, pos)
    _, dec_ref_bits = oracle.decode(b, k, enc_ref, pos_ref)
    assert np.array_equal(_bits(dec_gpu), dec_ref_bits)

    acc_gpu = torch.full((M, N), 12345, dtype=torch.int32, device=dev)
    out_gpu = sq.sq_gemm(fmt, enc_gpu, w_gpu, pos, acc_out=acc_gpu)
    check_status()
    if full_gemm:
        acc_ref, ref32, out_ref = oracle.gemm(b, k, enc_ref, w_ref, pos_ref)
        assert np.array_equal(_np(acc_gpu), acc_ref)
        assert_bf16_close(out_gpu, ref32)
        assert np.array_equal(_bits(out_gpu), out_ref)   # same IEEE ops, same order: equal in practice
    else:
        rng = np.random.default_rng(seed)
        rows = np.unique(np.concatenate([[0, M - 1], rng.integers(0, M, 24)]))
        cols = np.unique(np.concatenate([[0, N - 1], rng.integers(0, N, 96)]))
        acc_ref, ref32, out_ref = oracle.gemm(b, k, enc_ref, w_ref, pos_ref, rows=rows, cols=cols)
        assert np.array_equal(_np(acc_gpu)[np.ix_(rows, cols)], acc_ref)
        assert_bf16_close(out_gpu[rows][:, cols], ref32)
    # without the accumulator dump the bf16 output is the same
    out2 = sq.sq_gemm(fmt, enc_gpu, w_gpu, pos)
    assert torch.equal(out2, out_gpu)
    check_status()


# ----------------------------------------------------------------------------- small, ragged, multi-tile

@pytest.mark.parametrize("b,k,static", [
    (64, 8, False), (64, 8, True), (32, 2, False), (32, 8, True), (128, 16, True), (128, 8, False),
    (64, 16, False), (64, 4, True), (128, 32, False), (32, 1, False), (64, 32, True),
    # k not a power of two: rank-by-counting encode, byte-wise sparse merge in the GEMM, static
    # positions that TMA cannot fetch ((K/b)*k not a multiple of 16)
    (64, 12, False), (64, 12, True), (32, 3, False), (32, 3, True), (128, 24, False), (128, 24, True),
    (64, 5, False), (64, 5, True), (128, 7, False), (32, 15, True),
])
def test_small_ragged_shapes(b, k, static):
    # 2 M-tiles with a ragged tail, 2 N-tiles with a ragged tail, 3 K steps
    run_pipeline(M=200, N=328, K=384, b=b, k=k, static=static, seed=b + k)


@pytest.mark.parametrize("M", [1, 16, 127, 128, 129])
def test_row_counts_around_a_tile(M):
    run_pipeline(M=M, N=264, K=256, b=64, k=8, static=False, seed=M)


def test_deep_k_exceeds_the_pipeline_depth():
    # 12 K steps (> 2x the number of shared-memory stages), one tile
    run_pipeline(M=96, N=128, K=1536, b=64, k=8, static=False, seed=7)
    run_pipeline(M=96, N=128, K=1536, b=128, k=16, static=True, seed=8)


def test_config1_single_gemm():
    """M=64, K=N=4096, N(0,1) activations with 1% channels x20, b=64, k=8 dynamic."""
    run_pipeline(M=64, N=4096, K=4096, b=64, k=8, static=False, seed=0, dist="normal", frac=0.01, scale=20.0)


def test_degenerate_rows():
    """Zero rows, constant rows (every element ties), one-hot rows, and a row that clamps."""
    K, b, k = 256, 64, 8
    X = gen.activations(8, K, seed=3, device="cpu").float()
    X[0] = 0
    X[1] = -3.0
    X[2] = 0
    X[2, 77] = 2.5
    X[3, :] = 1.0
    X[3, 5] = 1.0078125          # barely above the ties
    X[4] = X[4].abs().clamp_min(0.5)   # all close to each other -> shift 4 and clamping
    X = X.to(torch.bfloat16).cuda()
    run_pipeline(M=8, N=64, K=K, b=b, k=k, static=False, X=X)
    run_pipeline(M=8, N=64, K=K, b=b, k=k, static=True, X=X)


def test_empty_problem_is_a_no_op():
    fmt = sq.make_format(64, 8, False)
    X = torch.empty(0, 256, dtype=torch.bfloat16, device="cuda")
    enc = sq.sq_encode(fmt, X)
    W = gen.weights(16, 256, device="cuda")
    w = sq.sq_pack_weights(fmt, W)
    out = sq.sq_gemm(fmt, enc, w)
    assert out.shape == (0, 16)
    assert sq.sq_decode(fmt, enc).shape == (0, 256)
    check_status()


def test_maximum_k():
    """K = SQ_MAX_K: the largest row the encoder stages and the largest accumulation depth."""
    K = sq.SQ_MAX_K
    b, k = 128, 16
    fmt = sq.make_format(b, k, False)
    X = gen.activations(4, K, seed=1, device="cuda")
    W = gen.weights(8, K, seed=1, device="cuda")
    enc = sq.sq_encode(fmt, X)
    w = sq.sq_pack_weights(fmt, W)
    acc = torch.zeros(4, 8, dtype=torch.int32, device="cuda")
    out = sq.sq_gemm(fmt, enc, w, acc_out=acc)
    check_status()
    enc_ref = oracle.encode(b, k, _bits(X))
    w_ref = oracle.pack_weights(b, k, _bits(W))
    compare_encoded(enc, enc_ref)
    acc_ref, ref32, _ = oracle.gemm(b, k, enc_ref, w_ref)
    assert np.array_equal(_np(acc), acc_ref)
    assert_bf16_close(out, ref32)


@pytest.mark.parametrize("b,k", [(128, 64), (32, 16), (64, 5)])
def test_maximum_k_static(b, k):
    """K = SQ_MAX_K with static positions, up to half of every bank selected: a row, its offset
    table and its stash no longer fit the staged kernels' shared memory, so the encoder has to pick
    a kernel that does; the GEMM walks 512 dense and up to 256 sparse K steps."""
    K = sq.SQ_MAX_K
    fmt = sq.make_format(b, k, True)
    X = gen.activations(5, K, seed=2, device="cuda")
    W = gen.weights(8, K, seed=2, device="cuda")
    calib = gen.calibration_batch(16, K, seed=2, device="cuda")
    pos = sq.sq_calib_positions(fmt, calib, W)
    pos_ref = oracle.calib_positions(b, k, _bits(calib), _bits(W))
    assert np.array_equal(_np(pos), pos_ref)
    enc = sq.sq_encode(fmt, X, pos)
    w = sq.sq_pack_weights(fmt, W, pos)
    acc = torch.zeros(5, 8, dtype=torch.int32, device="cuda")
    out = sq.sq_gemm(fmt, enc, w, pos, acc_out=acc)
    check_status()
    enc_ref = oracle.encode(b, k, _bits(X), pos_ref)
    w_ref = oracle.pack_weights(b, k, _bits(W), pos_ref)
    compare_encoded(enc, enc_ref)
    compare_weights(w, w_ref)
    acc_ref, ref32, _ = oracle.gemm(b, k, enc_ref, w_ref, pos_ref)
    assert np.array_equal(_np(acc), acc_ref)
    assert_bf16_close(out, ref32)


def test_worst_case_accumulator_magnitude():
    """All-maximal codes of one sign: the internal offset form must not overflow int32."""
    K, b, k = 8192, 64, 8
    fmt = sq.make_format(b, k, False)
    X = torch.full((2, K), 3.0, dtype=torch.bfloat16, device="cuda")
    X[1] = -3.0
    W = torch.full((8, K), 0.5, dtype=torch.bfloat16, device="cuda")
    W[1] = -0.5
    enc = sq.sq_encode(fmt, X)
    w = sq.sq_pack_weights(fmt, W)
    acc = torch.zeros(2, 8, dtype=torch.int32, device="cuda")
    sq.sq_gemm(fmt, enc, w, acc_out=acc)
    check_status()
    enc_ref = oracle.encode(b, k, _bits(X))
    w_ref = oracle.pack_weights(b, k, _bits(W))
    acc_ref, _, _ = oracle.gemm(b, k, enc_ref, w_ref)
    assert np.array_equal(_np(acc), acc_ref)
    # (K/b)*k entries at 127 and the rest at 7 << 4 = 112, times 7
    assert abs(int(acc_ref[0, 0])) == ((K // b) * k * 127 + (K - (K // b) * k) * 112) * 7


@pytest.mark.parametrize("M,N,K,b,k,static", [
    (128, 256 * 300, 1024, 64, 8, False),     # one CTA per tile: 300 tiles, two or three per SM, 8 K steps each
    (512, 256 * 160, 512, 128, 16, True),     # CTA pairs: whole tiles + a last wave cut in two, TMA-fed sparse K steps
    (640, 256 * 150, 768, 64, 8, False),      # CTA pairs: whole tiles, cut tiles and the odd last row unit together
    (512, 256 * 60, 384, 64, 8, True),        # CTA pairs: one wave of whole tiles (cutting would not save a wave)
    (257, 256 * 80, 256, 64, 8, False),       # CTA pairs: second row unit holds a single row
    (256, 256 * 90, 256, 32, 4, True),        # CTA pairs: exactly one row unit (only "odd unit" tiles)
    (1031, 264, 640, 128, 16, False),         # CTA pairs: ragged rows and a ragged, single column tile
])
def test_several_tiles_per_sm(M, N, K, b, k, static):
    """Persistent-kernel steady state: every SM walks through several tiles, so the pipelines
    wrap around tile boundaries.  Sampled token rows are checked over EVERY output channel."""
    fmt = sq.make_format(b, k, static)
    X = gen.activations(M, K, seed=11, device="cuda")
    W = gen.weights(N, K, seed=11, device="cuda")
    pos = pos_ref = None
    if static:
        pos = sq.sq_calib_positions(fmt, gen.calibration_batch(64, K, seed=11, device="cuda"))
        pos_ref = _np(pos)
    w = sq.sq_pack_weights(fmt, W, pos)
    enc = sq.sq_encode(fmt, X, pos)
    rows = np.unique(np.clip(np.concatenate([[0, 127, 128, M - 1], np.arange(5, M, max(M // 12, 1))]), 0, M - 1))
    enc_ref = oracle.encode(b, k, _bits(X)[rows], pos_ref)
    w_ref = oracle.pack_weights(b, k, _bits(W), pos_ref)
    acc_ref, ref32, _ = oracle.gemm(b, k, enc_ref, w_ref, pos_ref)
    for _ in range(3):                          # a race would not show on every launch
        acc = torch.empty(M, N, dtype=torch.int32, device="cuda")
        out = sq.sq_gemm(fmt, enc, w, pos, acc_out=acc)
        check_status()
        assert np.array_equal(_np(acc)[rows], acc_ref)
        assert_bf16_close(out[torch.from_numpy(rows).cuda()], ref32)


# ----------------------------------------------------------------------------- encode: static positions, staged rows / rows in registers

@pytest.mark.parametrize("K,b,k", [
    (2048, 64, 8), (4096, 32, 4), (4096, 128, 64), (6144, 64, 4), (7168, 128, 16),
    (12288, 64, 8), (14336, 64, 8), (16384, 32, 8), (24576, 128, 16), (32768, 64, 16),
])
def test_static_encode_row_slices_in_registers(K, b, k):
    """Static positions with rows of 1, 2, 4 or 8 warp slices (every slice size the kernels are
    built for), a ragged row count, and rows that are all zero, all ties, one-hot, and clamping."""
    M = 333
    fmt = sq.make_format(b, k, True)
    X = gen.activations(M, K, seed=K + k, outlier_fraction=0.01, outlier_scale=30.0, device="cpu").float()
    X[0] = 0
    X[1] = -3.0
    X[2] = 0
    X[2, K - 3] = 2.5
    X[3] = X[3].abs().clamp_min(0.5)
    X[M - 1] = 1.0
    X = X.to(torch.bfloat16).cuda()
    calib = gen.calibration_batch(64, K, seed=K, outlier_fraction=0.01, outlier_scale=30.0, device="cuda")
    pos = sq.sq_calib_positions(fmt, calib)
    pos_ref = oracle.calib_positions(b, k, _bits(calib))
    assert np.array_equal(_np(pos), pos_ref)
    enc = sq.sq_encode(fmt, X, pos)
    check_status()
    compare_encoded(enc, oracle.encode(b, k, _bits(X), pos_ref))


# ----------------------------------------------------------------------------- few rows: split-K through a workspace

@pytest.mark.parametrize("b,k,static", [
    (64, 8, False),     # producers merge (k/b = 1/8)
    (64, 16, False),    # epilogue warps merge, word path
    (32, 1, False),     # epilogue warps merge, byte path
    (128, 16, True),    # TMA-fed sparse K steps (the first part of K takes them all)
    (64, 4, True),
    (64, 12, False),    # k not a power of two: byte path
    (32, 3, True),
])
@pytest.mark.parametrize("M,K", [(1, 1024), (64, 2048), (128, 1536), (17, 4096)])
def test_split_k_with_workspace(b, k, static, M, K):
    """sq_gemm_ws with a workspace (K cut into parts + finishing kernel) against the oracle and,
    bit for bit, against the call without a workspace (K cut into parts that run as one
    thread-block cluster per column tile and add their partial sums through distributed shared
    memory)."""
    N = 520                       # three column tiles, the last one ragged
    fmt = sq.make_format(b, k, static)
    X = gen.activations(M, K, seed=M + K, outlier_fraction=0.01, outlier_scale=20.0, device="cuda")
    W = gen.weights(N, K, seed=K, device="cuda")
    pos = pos_ref = None
    if static:
        pos = sq.sq_calib_positions(fmt, gen.calibration_batch(64, K, seed=K, device="cuda"), W)
        pos_ref = _np(pos)
    w = sq.sq_pack_weights(fmt, W, pos)
    enc = sq.sq_encode(fmt, X, pos)
    need = sq.sq_gemm_workspace_bytes(fmt, M, N, K)
    if need == 0:
        # at most 64 rows in a format the weight-streaming kernel serves: no workspace is of use
        # (one that is passed anyway is ignored)
        assert M <= 64
        need = 8 * M * N * 4
    else:
        assert need % (M * N * 4) == 0 and need // (M * N * 4) in (2, 4, 8)
    ws = torch.full((need,), 0xAB, dtype=torch.uint8, device="cuda")     # stale contents must not matter
    acc = torch.empty(M, N, dtype=torch.int32, device="cuda")
    out = sq.sq_gemm_ws(fmt, enc, w, pos, acc_out=acc, workspace=ws)
    out_again = sq.sq_gemm_ws(fmt, enc, w, pos, workspace=ws).clone()
    acc1 = torch.empty(M, N, dtype=torch.int32, device="cuda")
    out1 = sq.sq_gemm_ws(fmt, enc, w, pos, acc_out=acc1, workspace=None)
    small = sq.sq_gemm_ws(fmt, enc, w, pos, workspace=ws[: 2 * M * N * 4]).clone()   # room for two parts only
    check_status()
    assert torch.equal(acc, acc1) and torch.equal(out, out1) and torch.equal(out_again, out1) and torch.equal(small, out1)
    enc_ref = oracle.encode(b, k, _bits(X), pos_ref)
    w_ref = oracle.pack_weights(b, k, _bits(W), pos_ref)
    acc_ref, ref32, out_ref = oracle.gemm(b, k, enc_ref, w_ref, pos_ref)
    assert np.array_equal(_np(acc), acc_ref)
    assert_bf16_close(out, ref32)
    assert np.array_equal(_bits(out), out_ref)


# ----------------------------------------------------------------------------- few rows: the weight-streaming kernel

@pytest.mark.parametrize("b,k,static", [(64, 8, False), (64, 16, False), (128, 16, False), (32, 16, False), (128, 64, False)])
@pytest.mark.parametrize("M,N,K", [(1, 136, 512), (16, 4096, 4096), (5, 1032, 1536), (13, 520, 2048), (16, 264, 14336),
                                   (16, 28672, 1024), (2, 8, 128), (9, 1160, 6144)])
def test_few_token_weight_streaming(b, k, static, M, N, K):
    """At most 16 rows: slabs of 128 output channels with the tokens as the narrow MMA operand, K in
    1, 2, 4 or 8 parts per slab that add their sums through distributed shared memory; ragged slabs,
    one to 224 slabs, static (TMA-fed sparse K steps) and dynamic (merged) positions."""
    fmt = sq.make_format(b, k, static)
    assert sq.sq_gemm_workspace_bytes(fmt, M, N, K) == 0
    X = gen.activations(M, K, seed=M + N, outlier_fraction=0.01, outlier_scale=20.0, device="cuda")
    W = gen.weights(N, K, seed=N + K, device="cuda")
    pos = pos_ref = None
    if static:
        pos = sq.sq_calib_positions(fmt, gen.calibration_batch(32, K, seed=K, device="cuda"), W)
        pos_ref = _np(pos)
    w = sq.sq_pack_weights(fmt, W, pos)
    enc = sq.sq_encode(fmt, X, pos)
    acc = torch.full((M, N), -7, dtype=torch.int32, device="cuda")
    out = sq.sq_gemm(fmt, enc, w, pos, acc_out=acc)
    again = sq.sq_gemm(fmt, enc, w, pos).clone()
    check_status()
    enc_ref = oracle.encode(b, k, _bits(X), pos_ref)
    w_ref = oracle.pack_weights(b, k, _bits(W), pos_ref)
    rng = np.random.default_rng(N)
    cols = None if N * K <= 1 << 24 else np.unique(np.concatenate([[0, 127, 128, N - 1], rng.integers(0, N, 600)]))
    acc_ref, ref32, out_ref = oracle.gemm(b, k, enc_ref, w_ref, pos_ref, cols=cols)
    sel = slice(None) if cols is None else cols
    assert np.array_equal(_np(acc)[:, sel], acc_ref)
    assert_bf16_close(out[:, sel] if cols is None else out[:, torch.from_numpy(cols).cuda()], ref32)
    assert np.array_equal(_bits(out)[:, sel], out_ref) and torch.equal(out, again)


# ----------------------------------------------------------------------------- many rows: pre-widened activations

@pytest.mark.parametrize("b,k,static", [(64, 8, False), (32, 1, False), (128, 64, False), (128, 16, True), (64, 4, True),
                                        (64, 12, False), (32, 3, True), (128, 24, False), (64, 5, True)])
@pytest.mark.parametrize("M,K", [(200, 384), (513, 1024), (300, 128)])
def test_prewidened_activations_with_workspace(b, k, static, M, K):
    """sq_gemm_ws with M*K bytes of workspace (activations expanded once into 8-bit tensor-core
    operands) against the oracle and, bit for bit, against the calls without or with too little
    workspace (which widen, and merge, inside the GEMM kernel)."""
    N = 1288                      # six column tiles, the last one ragged
    fmt = sq.make_format(b, k, static)
    X = gen.activations(M, K, seed=M + K, outlier_fraction=0.01, outlier_scale=20.0, device="cuda")
    W = gen.weights(N, K, seed=K, device="cuda")
    pos = pos_ref = None
    if static:
        pos = sq.sq_calib_positions(fmt, gen.calibration_batch(64, K, seed=K, device="cuda"), W)
        pos_ref = _np(pos)
    w = sq.sq_pack_weights(fmt, W, pos)
    enc = sq.sq_encode(fmt, X, pos)
    need = sq.sq_gemm_workspace_bytes(fmt, M, N, K)
    assert need == M * K
    ws = torch.full((need,), 0x5A, dtype=torch.uint8, device="cuda")
    acc = torch.empty(M, N, dtype=torch.int32, device="cuda")
    out = sq.sq_gemm_ws(fmt, enc, w, pos, acc_out=acc, workspace=ws)
    again = sq.sq_gemm_ws(fmt, enc, w, pos, workspace=ws).clone()
    acc0 = torch.empty(M, N, dtype=torch.int32, device="cuda")
    plain = sq.sq_gemm_ws(fmt, enc, w, pos, acc_out=acc0, workspace=None)
    short = sq.sq_gemm_ws(fmt, enc, w, pos, workspace=ws[: need - 16]).clone()
    check_status()
    assert torch.equal(acc, acc0) and torch.equal(out, plain) and torch.equal(again, plain) and torch.equal(short, plain)
    enc_ref = oracle.encode(b, k, _bits(X), pos_ref)
    w_ref = oracle.pack_weights(b, k, _bits(W), pos_ref)
    acc_ref, ref32, out_ref = oracle.gemm(b, k, enc_ref, w_ref, pos_ref)
    assert np.array_equal(_np(acc), acc_ref)
    assert_bf16_close(out, ref32)
    assert np.array_equal(_bits(out), out_ref)


# ----------------------------------------------------------------------------- independent scales (static positions)

@pytest.mark.parametrize("b,k", [(64, 8), (128, 16), (32, 8), (128, 64)])
@pytest.mark.parametrize("M,K", [(37, 2048), (5, 384), (130, 3584)])
def test_indep_encode_and_decode(b, k, M, K):
    """SQ_POS_STATIC_INDEP: encode (the register kernel for K = 2048 and 3584, the plain kernel for
    K = 384) and decode against the oracle, bit for bit."""
    fmt = sq.make_format(b, k, True, independent_scales=True)
    X = gen.activations(M, K, seed=M + K + b, outlier_fraction=0.01, outlier_scale=20.0, device="cuda")
    W = gen.weights(24, K, seed=K, device="cuda")
    pos = sq.sq_calib_positions(sq.make_format(b, k, True), gen.calibration_batch(64, K, seed=K, device="cuda"), W)
    enc = sq.sq_encode(fmt, X, pos)
    check_status()
    ref = oracle.encode_indep(b, k, _bits(X), _np(pos))
    compare_encoded(enc, ref)
    dec = sq.sq_decode(fmt, enc, pos)
    _, ref_bits = oracle.decode(b, k, ref, _np(pos))
    assert np.array_equal(_bits(dec), ref_bits)


def test_indep_encode_degenerate_rows():
    b, k, K = 64, 8, 2048
    fmt = sq.make_format(b, k, True, independent_scales=True)
    pos = torch.arange(k, dtype=torch.uint8, device="cuda").repeat(K // b, 1).contiguous()
    X = torch.zeros(4, K, dtype=torch.bfloat16, device="cuda")
    X[1, 3] = 5.0       # only a selected place
    X[2, 40] = -3.0     # only an unselected place
    X[3, 3], X[3, 40] = 1e-30, -1e30
    enc = sq.sq_encode(fmt, X, pos)
    check_status()
    compare_encoded(enc, oracle.encode_indep(b, k, _bits(X), _np(pos)))


@pytest.mark.parametrize("b,k", [(64, 8), (128, 16), (32, 4)])
@pytest.mark.parametrize("M,N,K", [(64, 264, 512), (200, 520, 1024), (513, 1288, 2048), (1, 8, 512)])
def test_indep_gemm(b, k, M, N, K):
    """Two accumulators (dense and sparse product) and the fp32 join, against the oracle: both
    integer sums and the bf16 bits exact; with and without a workspace argument."""
    fmt = sq.make_format(b, k, True, independent_scales=True)
    X = gen.activations(M, K, seed=M + N, outlier_fraction=0.01, outlier_scale=20.0, device="cuda")
    W = gen.weights(N, K, seed=N + K, device="cuda")
    pos = sq.sq_calib_positions(sq.make_format(b, k, True), gen.calibration_batch(64, K, seed=K, device="cuda"), W)
    w = sq.sq_pack_weights(fmt, W, pos)
    enc = sq.sq_encode(fmt, X, pos)
    assert sq.sq_gemm_workspace_bytes(fmt, M, N, K) == 0
    acc = torch.empty(2, M, N, dtype=torch.int32, device="cuda")
    out = sq.sq_gemm(fmt, enc, w, pos, acc_out=acc)
    ws = torch.empty(M * K, dtype=torch.uint8, device="cuda")
    out2 = sq.sq_gemm_ws(fmt, enc, w, pos, workspace=ws).clone()
    check_status()
    pos_ref = _np(pos)
    enc_ref = oracle.encode_indep(b, k, _bits(X), pos_ref)
    w_ref = oracle.pack_weights(b, k, _bits(W), pos_ref)
    compare_encoded(enc, enc_ref)
    compare_weights(w, w_ref)
    lo, hi, ref32, out_ref = oracle.gemm_indep(b, k, enc_ref, w_ref, pos_ref)
    assert np.array_equal(_np(acc[0]), lo) and np.array_equal(_np(acc[1]), hi)
    assert_bf16_close(out, ref32)
    assert np.array_equal(_bits(out), out_ref) and torch.equal(out, out2)


def test_indep_gemm_rejects_what_it_cannot_run():
    fmt = sq.make_format(32, 1, True, independent_scales=True)   # (K/b)*k = 8: not a multiple of 16
    M, N, K = 16, 64, 256
    X = gen.activations(M, K, seed=1, device="cuda")
    W = gen.weights(N, K, seed=1, device="cuda")
    pos = sq.sq_calib_positions(sq.make_format(32, 1, True), gen.calibration_batch(16, K, seed=1, device="cuda"), W)
    w = sq.sq_pack_weights(fmt, W, pos)
    enc = sq.sq_encode(fmt, X, pos)
    compare_encoded(enc, oracle.encode_indep(32, 1, _bits(X), _np(pos)))
    with pytest.raises(sq.SqError) as e:
        sq.sq_gemm(fmt, enc, w, pos)
    assert e.value.status == sq.SQ_ERR_UNSUPPORTED
    with pytest.raises(ValueError):
        sq.make_format(64, 8, False, independent_scales=True)


@pytest.mark.parametrize("static", [False, True])
@pytest.mark.parametrize("M,N,K", [(128, 8, 2048), (3, 264, 512), (100, 1032, 1024), (16, 2048, 4096)])
def test_few_rows_without_workspace(static, M, N, K):
    """Plain sq_gemm at M <= 128: K cut into parts that form one thread-block cluster per column
    tile (clusters of 2, 4 and 8; one, two, five and eight tiles, with ragged edges)."""
    b, k = 64, 8
    fmt = sq.make_format(b, k, static)
    X = gen.activations(M, K, seed=M + N, outlier_fraction=0.01, outlier_scale=20.0, device="cuda")
    W = gen.weights(N, K, seed=N + K, device="cuda")
    pos = pos_ref = None
    if static:
        pos = sq.sq_calib_positions(fmt, gen.calibration_batch(64, K, seed=K, device="cuda"), W)
        pos_ref = _np(pos)
    w = sq.sq_pack_weights(fmt, W, pos)
    enc = sq.sq_encode(fmt, X, pos)
    acc = torch.empty(M, N, dtype=torch.int32, device="cuda")
    out = sq.sq_gemm(fmt, enc, w, pos, acc_out=acc, use_workspace=False)
    again = sq.sq_gemm(fmt, enc, w, pos, use_workspace=False).clone()
    check_status()
    enc_ref = oracle.encode(b, k, _bits(X), pos_ref)
    w_ref = oracle.pack_weights(b, k, _bits(W), pos_ref)
    acc_ref, ref32, out_ref = oracle.gemm(b, k, enc_ref, w_ref, pos_ref)
    assert np.array_equal(_np(acc), acc_ref)
    assert_bf16_close(out, ref32)
    assert np.array_equal(_bits(out), out_ref) and torch.equal(out, again)


# ----------------------------------------------------------------------------- producer fusion (Section 3.3)

def merged_operand_from_oracle(b, k, enc_ref, pos_ref):
    """The product's merged 8-bit operand written out from the oracle's encoding: byte = code * 2^e + 128
    for a dense element, INT8 code + 128 for a selected one, stored in the tensor-core K order of one
    32-element block (16 even elements, then 16 odd)."""
    by = enc_ref.dq4.astype(np.int32)                              # element 2i in the low nibble, 2i+1 in the high one
    M, K = by.shape[0], by.shape[1] * 2
    dq = np.empty((M, K), dtype=np.int32)
    dq[:, 0::2] = ((by & 15) ^ 8) - 8
    dq[:, 1::2] = ((by >> 4) ^ 8) - 8
    merged = dq << enc_ref.shift.astype(np.int32)[:, None]
    G = K // b
    idx = enc_ref.idx if enc_ref.idx is not None else np.broadcast_to(pos_ref.reshape(1, G, k), (M, G, k))
    cols = (np.arange(G)[None, :, None] * b + idx.astype(np.int64)).reshape(M, G * k)
    np.put_along_axis(merged, cols, enc_ref.vals.reshape(M, G * k).astype(np.int32), axis=1)
    j = np.arange(K)
    where = 32 * (j // 32) + 16 * (j % 2) + (j % 32) // 2
    out = np.empty((M, K), dtype=np.uint8)
    out[:, where] = (merged + 128).astype(np.uint8)
    return out


@pytest.mark.parametrize("M,N,K,b,k,static", [
    (300, 1024, 2048, 64, 8, True),      # rows staged in shared-memory slots, one warp per row
    (257, 1280, 8192, 64, 8, True),      # ... rows split over two warps
    (40, 256, 28672, 128, 16, True),     # ... long rows: eight warps per row, byte masks
    (20, 256, 32768, 64, 8, True),       # slots, tables and image do not fit: the register kernel
    (200, 1024, 4096, 128, 16, True),
    (130, 1024, 3072, 32, 4, True),
    (140, 1024, 2048, 64, 6, True),      # k not a multiple of four: byte-wise sparse path
    (150, 1024, 1024, 64, 8, True),      # row length the register kernel does not take: second kernel
    (200, 1024, 2048, 64, 8, False),     # dynamic positions: second kernel
    (40, 512, 2048, 64, 8, True),        # few rows: the product ignores the merged operand
])
def test_encode_with_merged_operand(M, N, K, b, k, static):
    dev = "cuda"
    fmt = sq.make_format(b, k, static)
    X = gen.activations(M, K, seed=5, device=dev)
    W = gen.weights(N, K, seed=5, device=dev)
    pos = pos_ref = None
    if static:
        calib = gen.calibration_batch(64, K, seed=5, device=dev)
        pos = sq.sq_calib_positions(fmt, calib, W)
        pos_ref = _np(pos)
    enc_ref = oracle.encode(b, k, _bits(X), pos_ref)
    a8 = torch.full((M, K), 0x5A, dtype=torch.uint8, device=dev)
    enc_gpu, a8 = sq.sq_encode_a8(fmt, X, pos, a8=a8)
    check_status()
    compare_encoded(enc_gpu, enc_ref)
    assert np.array_equal(_np(a8), merged_operand_from_oracle(b, k, enc_ref, pos_ref))

    w_gpu = sq.sq_pack_weights(fmt, W, pos)
    w_ref = oracle.pack_weights(b, k, _bits(W), pos_ref)
    keep = a8.clone()
    acc_gpu = torch.full((M, N), -7, dtype=torch.int32, device=dev)
    out_gpu = sq.sq_gemm_a8(fmt, enc_gpu, a8, w_gpu, pos, acc_out=acc_gpu)
    check_status()
    assert torch.equal(a8, keep)                       # read, never written
    acc_ref, ref32, out_ref = oracle.gemm(b, k, enc_ref, w_ref, pos_ref)
    assert np.array_equal(_np(acc_gpu), acc_ref)
    assert np.array_equal(_bits(out_gpu), out_ref)
    assert torch.equal(sq.sq_gemm(fmt, enc_gpu, w_gpu, pos), out_gpu)


def test_merged_operand_rejects_independent_scales():
    fmt = sq.make_format(64, 8, True, independent_scales=True)
    X = gen.activations(8, 1024, seed=1, device="cuda")
    pos = torch.arange(8, dtype=torch.uint8, device="cuda").repeat(1024 // 64)
    with pytest.raises(sq.SqError):
        sq.sq_encode_a8(fmt, X, pos)


# ----------------------------------------------------------------------------- measurement aid

def test_tensor_rate_probe_runs_and_counts_its_operations():
    """The probe issues iterations x 128 x 256 x 128 multiply-adds on every SM, leaves the status word
    alone and hands tensor memory back (a product call right after it works)."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    ops = sq.sq_probe_int8_tensor_rate(500)
    torch.cuda.synchronize()
    assert ops == 2.0 * 128 * 256 * 128 * 500 * sms
    check_status()
    with pytest.raises(sq.SqError):
        sq.sq_probe_int8_tensor_rate(0)
    run_pipeline(M=96, N=128, K=256, b=64, k=8, static=False, seed=11)


def test_fp8_tensor_rate_probe_runs_and_counts_its_operations():
    """The floating-point variant's probe: the same count, the status word clean, tensor memory handed back."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    ops = sq.sq_probe_fp8_tensor_rate(500)
    torch.cuda.synchronize()
    assert ops == 2.0 * 128 * 256 * 128 * 500 * sms
    check_status()
    with pytest.raises(sq.SqError):
        sq.sq_probe_fp8_tensor_rate(0)
    run_pipeline(M=96, N=128, K=256, b=64, k=8, static=False, seed=12)


# ----------------------------------------------------------------------------- few-token product started early

def test_few_token_product_in_a_chain_reads_what_its_predecessor_wrote():
    """The few-token product may start while the encode before it on the stream still runs (it only
    fetches weights until that one has completed).  Chains of encode -> product over changing
    inputs, issued back to back on one stream and replayed from a CUDA graph, must give what the
    calls give one at a time: the product never sees the previous tokens' codes, scales or shifts,
    and the next encode never overwrites them under a product that still reads them."""
    fmt = sq.make_format(64, 8, False)
    M, K, N = 16, 4096, 1032
    W = gen.weights(N, K, seed=21, device="cuda")
    w = sq.sq_pack_weights(fmt, W)
    Xs = [gen.activations(M, K, seed=100 + i, outlier_fraction=0.01, outlier_scale=float(5 * (i + 1)), device="cuda") for i in range(6)]
    # one at a time, with a synchronisation after every call
    want = []
    for X in Xs:
        enc = sq.sq_encode(fmt, X)
        torch.cuda.synchronize()
        want.append(sq.sq_gemm(fmt, enc, w).clone())
        torch.cuda.synchronize()
    # back to back: ONE encoding buffer reused by every link of the chain
    enc = sq.alloc_encoded(fmt, M, K, "cuda")
    outs = [torch.empty(M, N, dtype=torch.bfloat16, device="cuda") for _ in Xs]

    def chain():
        for X, out in zip(Xs, outs):
            sq.sq_encode(fmt, X, out=enc)
            sq.sq_gemm(fmt, enc, w, out=out)
    for _ in range(3):
        for out in outs:
            out.zero_()
        chain()
        torch.cuda.synchronize()
        for got, ref in zip(outs, want):
            assert torch.equal(got, ref)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            chain()
    for _ in range(3):
        for out in outs:
            out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        for got, ref in zip(outs, want):
            assert torch.equal(got, ref)
    check_status()
    # ... and the first of them against the oracle
    enc_ref = oracle.encode(64, 8, _bits(Xs[0]))
    _, _, out_ref = oracle.gemm(64, 8, enc_ref, oracle.pack_weights(64, 8, _bits(W)))
    assert np.array_equal(_bits(want[0]), out_ref)


@pytest.mark.parametrize("b,k", [(64, 8), (128, 16), (32, 4), (64, 32)])
@pytest.mark.parametrize("M,K", [(1, 4096), (5, 14336), (16, 4096), (100, 14336), (148, 2048), (149, 4096), (300, 14336),
                                 (37, 28672), (130, 8192)])
def test_encode_few_rows_many_warps_per_row(b, k, M, K):
    """Few rows: the encoder gives a row up to sixteen warps (every row a group of its own, all rows
    in one wave of blocks) instead of packing many one-warp rows into a block; dynamic positions and
    the static ones of row lengths the staged-row kernels leave to it."""
    X = gen.activations(M, K, seed=M + K + b, outlier_fraction=0.01, outlier_scale=25.0, device="cuda")
    fmt = sq.make_format(b, k, False)
    enc = sq.sq_encode(fmt, X)
    check_status()
    compare_encoded(enc, oracle.encode(b, k, _bits(X)))
    dec = sq.sq_decode(fmt, enc)
    assert np.array_equal(_bits(dec), oracle.decode(b, k, oracle.encode(b, k, _bits(X)))[1])


@pytest.mark.parametrize("b,k", [(64, 8), (128, 16), (32, 4), (64, 16)])
@pytest.mark.parametrize("M,N,K", [(1, 520, 1024), (16, 264, 2048), (5, 1032, 4096), (3, 520, 14336), (16, 8, 512), (9, 4104, 4096)])
def test_few_tokens_static_positions_on_the_weight_streaming_kernel(b, k, M, N, K):
    """At most 16 tokens with STATIC positions: the weight-streaming kernel merges the sparse entries
    at the places of one shared row of positions (a per-token row of them for dynamic positions)."""
    run_pipeline(M=M, N=N, K=K, b=b, k=k, static=True, seed=M + N + K)


@pytest.mark.parametrize("static", [False, True])
@pytest.mark.parametrize("b,k", [(64, 8), (128, 16), (32, 4), (64, 32)])
@pytest.mark.parametrize("M,N,K", [(17, 264, 1024), (32, 1032, 4096), (25, 520, 14336), (33, 264, 2048), (48, 4104, 4096),
                                   (64, 136, 1536), (64, 19080, 1024)])
def test_up_to_64_tokens_on_the_weight_streaming_kernel(b, k, static, M, N, K):
    """17..32 and 33..64 tokens: the weight-streaming kernel with 32 / 64 accumulator columns (two
    issuing threads, one CTA per SM); the last shape has more slabs of 128 channels than SMs, which
    sends 33..64 tokens to the tiled kernel instead."""
    run_pipeline(M=M, N=N, K=K, b=b, k=k, static=static, seed=M + N + K + b)
