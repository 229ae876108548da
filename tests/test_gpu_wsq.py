"""Parity of weights in SQ-format (Algorithm 1's format) with the CPU oracle, through the C ABI:
codes, the implicit mask, compact values, both scales, the INT8 activations and both integer sums
bit-exact; bf16 outputs equal (the fp32 join is the same three IEEE operations on both sides)."""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2512_05409_b200 as sq

pytestmark = pytest.mark.gpu


def _np(t):
    return t.detach().cpu().numpy()


def _importance(W, seed):
    g = torch.Generator().manual_seed(seed)
    return (W.float().cpu() ** 2 * (0.2 + 4.8 * torch.rand(W.shape, generator=g))).contiguous().cuda()


def _unorder(xq_gpu):
    """Undo the product kernel's element order ([4 even | 4 odd] per 8)."""
    M, K = xq_gpu.shape
    x = xq_gpu.reshape(M, K // 8, 2, 4)            # [.., parity, i]
    return np.stack([x[:, :, 0, :], x[:, :, 1, :]], axis=-1).reshape(M, K)


@pytest.mark.parametrize("b,k", [(64, 8), (32, 4), (128, 16), (64, 5), (128, 64)])
@pytest.mark.parametrize("M,N,K", [(1, 264, 512), (4, 1032, 2048), (3, 8, 128), (2, 520, 4096)])
def test_weights_in_sq_format(b, k, M, N, K):
    fmt = sq.make_format(b, k, True)
    W = gen.weights(N, K, seed=N + K, device="cuda")
    X = gen.activations(M, K, seed=M + K, outlier_fraction=0.01, outlier_scale=20.0, device="cuda")
    imp = _importance(W, seed=b + k)
    imp[1] = 1.0                                       # a channel of all-equal scores: lower indices win
    enc = sq.sq_w_encode(fmt, W, imp)
    xq, s_x = sq.sq_w_act_quant(X)
    acc = torch.full((2, M, N), 7, dtype=torch.int32, device="cuda")
    out = sq.sq_w_gemm(fmt, xq, s_x, enc, acc_out=acc)
    out2 = sq.sq_w_gemm(fmt, xq, s_x, enc)
    assert sq.sq_device_status() == sq.SQ_OK and torch.equal(out, out2)
    ref = oracle.w_encode(b, k, gen.bf16_bits(W), _np(imp))
    assert np.array_equal(_np(enc.wq4), ref.wq4) and np.array_equal(_np(enc.w_hi), ref.w_hi)
    assert np.array_equal(_np(enc.s_high).view(np.uint32), ref.s_high.view(np.uint32))
    assert np.array_equal(_np(enc.s_low).view(np.uint32), ref.s_low.view(np.uint32))
    xq_ref, sx_ref = oracle.act_quant8(gen.bf16_bits(X))
    assert np.array_equal(_unorder(_np(xq)), xq_ref) and np.array_equal(_np(s_x).view(np.uint32), sx_ref.view(np.uint32))
    lo, hi, ref32, out_ref = oracle.w_gemm(b, k, xq_ref, sx_ref, ref)
    assert np.array_equal(_np(acc[0]), lo) and np.array_equal(_np(acc[1]), hi)
    assert np.array_equal(gen.bf16_bits(out), out_ref)
    got = out.float().cpu().numpy().astype(np.float64)
    nz = ref32 != 0
    assert np.all(np.abs(got[nz] - ref32[nz]) <= 1e-2 * np.abs(ref32[nz]))


@pytest.mark.parametrize("K,N", [(4096, 6144), (4096, 4096), (4096, 28672), (14336, 4096)])
def test_weights_in_sq_format_8b_shapes(K, N):
    """The 8B-decoder linears the benchmark times (b = 64, k = 8; 1 and 4 tokens): channels are
    independent, so the oracle recomputes sampled output channels from the same inputs."""
    b, k = 64, 8
    fmt = sq.make_format(b, k, True)
    W = gen.weights(N, K, seed=K + N, device="cuda")
    imp = (W.float() ** 2).contiguous()
    enc = sq.sq_w_encode(fmt, W, imp)
    rng = np.random.default_rng(K + N)
    ch = np.unique(np.concatenate([[0, 1, N - 2, N - 1], rng.integers(0, N, 200)]))
    ch_t = torch.from_numpy(ch).cuda()
    ref = oracle.w_encode(b, k, gen.bf16_bits(W[ch_t]), _np(imp[ch_t]))
    assert np.array_equal(_np(enc.wq4[ch_t]), ref.wq4) and np.array_equal(_np(enc.w_hi[ch_t]), ref.w_hi)
    assert np.array_equal(_np(enc.s_high[ch_t]).view(np.uint32), ref.s_high.view(np.uint32))
    assert np.array_equal(_np(enc.s_low[ch_t]).view(np.uint32), ref.s_low.view(np.uint32))
    for M in (1, 4):
        X = gen.activations(M, K, seed=M, outlier_fraction=0.01, outlier_scale=20.0, device="cuda")
        xq, s_x = sq.sq_w_act_quant(X)
        acc = torch.empty(2, M, N, dtype=torch.int32, device="cuda")
        out = sq.sq_w_gemm(fmt, xq, s_x, enc, acc_out=acc)
        assert sq.sq_device_status() == sq.SQ_OK
        xq_ref, sx_ref = oracle.act_quant8(gen.bf16_bits(X))
        assert np.array_equal(_unorder(_np(xq)), xq_ref)
        lo, hi, ref32, out_ref = oracle.w_gemm(b, k, xq_ref, sx_ref, ref)
        assert np.array_equal(_np(acc[0][:, ch_t]), lo) and np.array_equal(_np(acc[1][:, ch_t]), hi)
        assert np.array_equal(gen.bf16_bits(out[:, ch_t].contiguous()), out_ref)


def test_more_than_four_tokens_is_refused():
    fmt = sq.make_format(64, 8, True)
    W = gen.weights(8, 256, seed=1, device="cuda")
    enc = sq.sq_w_encode(fmt, W, torch.ones_like(W, dtype=torch.float32))
    xq, s_x = sq.sq_w_act_quant(gen.activations(5, 256, seed=1, device="cuda"))
    with pytest.raises(sq.SqError) as e:
        sq.sq_w_gemm(fmt, xq, s_x, enc)
    assert e.value.status == sq.SQ_ERR_UNSUPPORTED
