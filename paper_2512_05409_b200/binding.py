"""Thin ctypes binding of the C-ABI library (argument marshalling only).

Every function has the name and the argument order of its C counterpart in
`include/sq.h`; tensors are torch CUDA tensors whose `data_ptr()` is handed over,
and the stream is torch's current stream unless one is given.  Nothing is computed
here: every step of the path runs in the library's kernels.  There is no CPU
fallback -- if the library cannot be loaded the import fails.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

from . import build as _build

SQ_OK = 0
SQ_ERR_INVALID_ARG = 1
SQ_ERR_UNSUPPORTED = 2
SQ_ERR_NULL_POINTER = 3
SQ_ERR_ALIGNMENT = 4
SQ_ERR_ARCH = 5
SQ_ERR_CUDA = 6
SQ_ERR_TIMEOUT = 7

SQ_POS_DYNAMIC = 0
SQ_POS_STATIC = 1
SQ_POS_STATIC_INDEP = 2
SQ_LAYOUT_VERSION = 1
SQ_MAX_K = 65536


class sq_format(ctypes.Structure):
    _fields_ = [("bank", ctypes.c_int32), ("k", ctypes.c_int32),
                ("pos_mode", ctypes.c_int32), ("version", ctypes.c_int32)]


class sq_encoded(ctypes.Structure):
    _fields_ = [("dq4", ctypes.c_void_p), ("vals", ctypes.c_void_p), ("idx", ctypes.c_void_p),
                ("s_hi", ctypes.c_void_p), ("s_lo", ctypes.c_void_p), ("shift", ctypes.c_void_p)]


class sq_weights(ctypes.Structure):
    _fields_ = [("wq4", ctypes.c_void_p), ("s_w", ctypes.c_void_p), ("colsum", ctypes.c_void_p),
                ("w_sparse", ctypes.c_void_p)]


class SqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {sq_status_string(status)} (status {status})")


def _load() -> ctypes.CDLL:
    path = _build.LIB
    if _build.needs_build():
        path = _build.build()          # raises if nvcc is missing or the build fails
    lib = ctypes.CDLL(path)
    P, I64, VP = ctypes.POINTER, ctypes.c_int64, ctypes.c_void_p
    lib.sq_status_string.restype = ctypes.c_char_p
    lib.sq_status_string.argtypes = [ctypes.c_int]
    lib.sq_encoded_sizes.argtypes = [P(sq_format), I64, I64, P(ctypes.c_size_t)]
    lib.sq_weights_sizes.argtypes = [P(sq_format), I64, I64, P(ctypes.c_size_t)]
    lib.sq_calib_positions.argtypes = [P(sq_format), VP, I64, I64, VP, I64, VP, VP]
    lib.sq_pack_weights.argtypes = [P(sq_format), VP, I64, I64, VP, P(sq_weights), VP]
    lib.sq_encode.argtypes = [P(sq_format), VP, I64, I64, VP, P(sq_encoded), VP]
    lib.sq_gemm.argtypes = [P(sq_format), P(sq_encoded), P(sq_weights), VP, I64, I64, I64, VP, VP, VP]
    lib.sq_gemm_ws.argtypes = [P(sq_format), P(sq_encoded), P(sq_weights), VP, I64, I64, I64, VP, VP, VP,
                               ctypes.c_size_t, VP]
    lib.sq_encode_a8.argtypes = [P(sq_format), VP, I64, I64, VP, P(sq_encoded), VP, VP]
    lib.sq_rmsnorm_encode.argtypes = [P(sq_format), VP, VP, ctypes.c_float, I64, I64, VP, P(sq_encoded), VP, VP]
    lib.sq_gemm_a8.argtypes = [P(sq_format), P(sq_encoded), P(sq_weights), VP, I64, I64, I64, VP, VP, VP, VP]
    lib.sq_gemm_workspace_bytes.argtypes = [P(sq_format), I64, I64, I64, P(ctypes.c_size_t)]
    lib.sq_gemm_static_scratch.argtypes = [P(sq_format), P(sq_encoded), P(sq_weights), VP, I64, I64, I64, VP, VP, VP]
    lib.sq_decode.argtypes = [P(sq_format), P(sq_encoded), VP, I64, I64, VP, VP]
    lib.sq_device_status.argtypes = [VP]
    lib.sq_probe_int8_tensor_rate.argtypes = [ctypes.c_int, P(ctypes.c_double), VP]
    lib.sq_probe_fp8_tensor_rate.argtypes = [ctypes.c_int, P(ctypes.c_double), VP]
    lib.sq_fp_pack_weights.argtypes = [VP, I64, I64, VP, VP, VP, VP]
    lib.sq_fp_encode.argtypes = [P(sq_format), VP, I64, I64, VP, P(sq_encoded), VP, VP]
    lib.sq_fp_rmsnorm_encode.argtypes = [P(sq_format), VP, VP, ctypes.c_float, I64, I64, VP, P(sq_encoded), VP, VP]
    lib.sq_fp_gemm.argtypes = [VP, VP, VP, VP, I64, I64, I64, VP, VP, VP]
    lib.sq_fp_decode.argtypes = [P(sq_format), P(sq_encoded), VP, I64, I64, VP, VP]
    lib.sq_w_encode.argtypes = [P(sq_format), VP, VP, I64, I64, VP, VP, VP, VP, VP]
    lib.sq_w_act_quant.argtypes = [VP, I64, I64, VP, VP, VP]
    lib.sq_w_gemm.argtypes = [P(sq_format), VP, VP, VP, VP, VP, VP, I64, I64, I64, VP, VP, VP]
    lib.sq_device_status_word.argtypes = [P(VP)]
    for name in ("sq_encoded_sizes", "sq_weights_sizes", "sq_calib_positions", "sq_pack_weights",
                 "sq_encode", "sq_gemm", "sq_gemm_ws", "sq_gemm_workspace_bytes", "sq_gemm_static_scratch", "sq_decode",
                 "sq_device_status", "sq_device_status_word", "sq_fp_pack_weights", "sq_fp_encode", "sq_fp_gemm",
                 "sq_fp_decode", "sq_w_encode", "sq_w_act_quant", "sq_w_gemm", "sq_encode_a8", "sq_gemm_a8", "sq_rmsnorm_encode", "sq_fp_rmsnorm_encode",
                 "sq_probe_int8_tensor_rate", "sq_probe_fp8_tensor_rate"):
        getattr(lib, name).restype = ctypes.c_int
    return lib


_lib = _load()
LIBRARY_PATH = _build.LIB


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream(stream):
    """The CUDA stream handle to launch on: the given torch stream (or raw handle), else torch's
    current stream on the current device (the direct lookup is several times cheaper than building
    a torch.cuda.Stream object, which matters for decode-sized calls)."""
    if stream is None:
        if _raw_stream is not None:
            return ctypes.c_void_p(_raw_stream(torch.cuda.current_device()))
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _check(status: int, where: str):
    if status != SQ_OK:
        raise SqError(status, where)


def make_format(bank: int, k: int, static: bool, independent_scales: bool = False) -> sq_format:
    """independent_scales (static positions only): the two parts get their own per-token scales
    (SQ_POS_STATIC_INDEP) instead of scales tied by a power of two."""
    if independent_scales and not static:
        raise ValueError("independent scales are built for static positions")
    mode = SQ_POS_STATIC_INDEP if independent_scales else (SQ_POS_STATIC if static else SQ_POS_DYNAMIC)
    return sq_format(bank, k, mode, SQ_LAYOUT_VERSION)


@dataclass
class Encoded:
    """Torch-owned buffers of one sq_encoded (idx is None for static positions)."""
    dq4: torch.Tensor
    vals: torch.Tensor
    idx: torch.Tensor | None
    s_hi: torch.Tensor
    s_lo: torch.Tensor
    shift: torch.Tensor

    def c_struct(self) -> sq_encoded:
        return sq_encoded(self.dq4.data_ptr(), self.vals.data_ptr(),
                          self.idx.data_ptr() if self.idx is not None else None,
                          self.s_hi.data_ptr(), self.s_lo.data_ptr(), self.shift.data_ptr())


@dataclass
class Weights:
    """Torch-owned buffers of one sq_weights (w_sparse is None for dynamic positions)."""
    wq4: torch.Tensor
    s_w: torch.Tensor
    colsum: torch.Tensor
    w_sparse: torch.Tensor | None

    def c_struct(self) -> sq_weights:
        return sq_weights(self.wq4.data_ptr(), self.s_w.data_ptr(), self.colsum.data_ptr(),
                          self.w_sparse.data_ptr() if self.w_sparse is not None else None)


def sq_status_string(status: int) -> str:
    return _lib.sq_status_string(int(status)).decode()


def sq_encoded_sizes(fmt: sq_format, M: int, K: int) -> list[int]:
    out = (ctypes.c_size_t * 6)()
    _check(_lib.sq_encoded_sizes(ctypes.byref(fmt), M, K, out), "sq_encoded_sizes")
    return list(out)


def sq_weights_sizes(fmt: sq_format, N: int, K: int) -> list[int]:
    out = (ctypes.c_size_t * 4)()
    _check(_lib.sq_weights_sizes(ctypes.byref(fmt), N, K, out), "sq_weights_sizes")
    return list(out)


def _buf(nbytes: int, dtype, device):
    # at least 16 bytes so that an empty tensor still has a valid, aligned pointer
    n = max(nbytes, 16) // torch.empty((), dtype=dtype).element_size()
    return torch.empty(n, dtype=dtype, device=device)


def alloc_encoded(fmt: sq_format, M: int, K: int, device="cuda") -> Encoded:
    sz = sq_encoded_sizes(fmt, M, K)
    gk = (K // fmt.bank) * fmt.k
    dq4 = _buf(sz[0], torch.uint8, device)[: sz[0]].view(M, K // 2)
    vals = _buf(sz[1], torch.int8, device)[: sz[1]].view(M, K // fmt.bank, fmt.k)
    idx = None
    if fmt.pos_mode == SQ_POS_DYNAMIC:
        idx = _buf(sz[2], torch.uint8, device)[: sz[2]].view(M, K // fmt.bank, fmt.k)
    s_hi = _buf(sz[3], torch.float32, device)[:M]
    s_lo = _buf(sz[4], torch.float32, device)[:M]
    shift = _buf(sz[5], torch.uint8, device)[:M]
    assert gk * M == sz[1]
    return Encoded(dq4, vals, idx, s_hi, s_lo, shift)


def alloc_weights(fmt: sq_format, N: int, K: int, device="cuda") -> Weights:
    sz = sq_weights_sizes(fmt, N, K)
    wq4 = _buf(sz[0], torch.uint8, device)[: sz[0]].view(N, K // 2)
    s_w = _buf(sz[1], torch.float32, device)[:N]
    colsum = _buf(sz[2], torch.int32, device)[:N]
    w_sparse = None
    if fmt.pos_mode != SQ_POS_DYNAMIC:
        w_sparse = _buf(sz[3], torch.int8, device)[: sz[3]].view(N, (K // fmt.bank) * fmt.k)
    return Weights(wq4, s_w, colsum, w_sparse)


def _bf16_2d(t: torch.Tensor, name: str):
    if t.dtype != torch.bfloat16 or t.dim() != 2 or not t.is_contiguous() or not t.is_cuda:
        raise ValueError(f"{name} must be a contiguous 2-D CUDA bf16 tensor")
    return t.shape


def sq_calib_positions(fmt: sq_format, calib: torch.Tensor, W: torch.Tensor | None = None,
                       positions: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    T, K = _bf16_2d(calib, "calib")
    N = 0
    if W is not None:
        N, K2 = _bf16_2d(W, "W")
        if K2 != K:
            raise ValueError("calib and W disagree on K")
    if positions is None:
        positions = _buf(max(K // fmt.bank, 1) * fmt.k, torch.uint8, calib.device)[: (K // fmt.bank) * fmt.k]
        positions = positions.view(K // fmt.bank, fmt.k)
    _check(_lib.sq_calib_positions(ctypes.byref(fmt), _ptr(calib), T, K, _ptr(W), N, _ptr(positions),
                                   _stream(stream)), "sq_calib_positions")
    return positions


def sq_pack_weights(fmt: sq_format, W: torch.Tensor, positions: torch.Tensor | None = None,
                    out: Weights | None = None, stream=None) -> Weights:
    N, K = _bf16_2d(W, "W")
    if out is None:
        out = alloc_weights(fmt, N, K, W.device)
    cs = out.c_struct()
    _check(_lib.sq_pack_weights(ctypes.byref(fmt), _ptr(W), N, K, _ptr(positions), ctypes.byref(cs),
                                _stream(stream)), "sq_pack_weights")
    return out


def sq_encode(fmt: sq_format, X: torch.Tensor, positions: torch.Tensor | None = None,
              out: Encoded | None = None, stream=None) -> Encoded:
    M, K = _bf16_2d(X, "X")
    if out is None:
        out = alloc_encoded(fmt, M, K, X.device)
    cs = out.c_struct()
    _check(_lib.sq_encode(ctypes.byref(fmt), _ptr(X), M, K, _ptr(positions), ctypes.byref(cs),
                          _stream(stream)), "sq_encode")
    return out


def sq_encode_a8(fmt: sq_format, X: torch.Tensor, positions: torch.Tensor | None = None,
                 out: Encoded | None = None, a8: torch.Tensor | None = None, stream=None):
    """sq_encode that also writes the product's merged 8-bit operand; returns (Encoded, a8 uint8 [M, K])."""
    M, K = _bf16_2d(X, "X")
    if out is None:
        out = alloc_encoded(fmt, M, K, X.device)
    if a8 is None:
        a8 = _buf(M * K, torch.uint8, X.device)[: M * K].view(M, K)
    cs = out.c_struct()
    _check(_lib.sq_encode_a8(ctypes.byref(fmt), _ptr(X), M, K, _ptr(positions), ctypes.byref(cs), _ptr(a8),
                             _stream(stream)), "sq_encode_a8")
    return out, a8



def sq_rmsnorm_encode(fmt: sq_format, X: torch.Tensor, gamma: torch.Tensor, eps: float,
                      positions: torch.Tensor, out: Encoded | None = None, a8: torch.Tensor | None = None,
                      want_a8: bool = True, stream=None):
    """Root-mean-square normalisation fused into the static-position encode; returns (Encoded, a8 or None)."""
    M, K = _bf16_2d(X, "X")
    if gamma.dtype != torch.bfloat16 or gamma.numel() != K or not gamma.is_contiguous():
        raise ValueError("gamma must be a contiguous bf16 tensor of K elements")
    if out is None:
        out = alloc_encoded(fmt, M, K, X.device)
    if a8 is None and want_a8:
        a8 = _buf(M * K, torch.uint8, X.device)[: M * K].view(M, K)
    cs = out.c_struct()
    _check(_lib.sq_rmsnorm_encode(ctypes.byref(fmt), _ptr(X), _ptr(gamma), ctypes.c_float(eps), M, K, _ptr(positions),
                                  ctypes.byref(cs), _ptr(a8), _stream(stream)), "sq_rmsnorm_encode")
    return out, a8


def sq_gemm_a8(fmt: sq_format, A: Encoded, a8: torch.Tensor, W: Weights, positions: torch.Tensor | None = None,
               out: torch.Tensor | None = None, acc_out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """sq_gemm reading the merged operand sq_encode_a8 wrote for A."""
    M, K = A.dq4.shape[0], A.dq4.shape[1] * 2
    N = W.wq4.shape[0]
    if out is None:
        out = _buf(M * N * 2, torch.bfloat16, A.dq4.device)[: M * N].view(M, N)
    ca, cw = A.c_struct(), W.c_struct()
    _check(_lib.sq_gemm_a8(ctypes.byref(fmt), ctypes.byref(ca), ctypes.byref(cw), _ptr(positions), M, N, K,
                           _ptr(out), _ptr(acc_out), _ptr(a8), _stream(stream)), "sq_gemm_a8")
    return out


def sq_gemm_workspace_bytes(fmt: sq_format, M: int, N: int, K: int) -> int:
    need = ctypes.c_size_t(0)
    _check(_lib.sq_gemm_workspace_bytes(ctypes.byref(fmt), M, N, K, ctypes.byref(need)), "sq_gemm_workspace_bytes")
    return int(need.value)


def sq_gemm_ws(fmt: sq_format, A: Encoded, W: Weights, positions: torch.Tensor | None = None,
               out: torch.Tensor | None = None, acc_out: torch.Tensor | None = None,
               workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    M, K = A.dq4.shape[0], A.dq4.shape[1] * 2
    N = W.wq4.shape[0]
    if out is None:
        out = _buf(M * N * 2, torch.bfloat16, A.dq4.device)[: M * N].view(M, N)
    ca, cw = A.c_struct(), W.c_struct()
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.sq_gemm_ws(ctypes.byref(fmt), ctypes.byref(ca), ctypes.byref(cw), _ptr(positions), M, N, K,
                           _ptr(out), _ptr(acc_out), _ptr(workspace), nbytes, _stream(stream)), "sq_gemm_ws")
    return out


SQ_STATIC_SCRATCH_BYTES = 16 << 20


def sq_gemm_static_scratch(fmt: sq_format, A: Encoded, W: Weights, positions: torch.Tensor | None = None,
                           out: torch.Tensor | None = None, acc_out: torch.Tensor | None = None,
                           stream=None) -> torch.Tensor:
    """The C ABI's sq_gemm_static_scratch: few-row GEMM whose split-K scratch is a fixed array inside
    the library, for callers that may not allocate device memory at call time.  `out` should be given
    by such a caller: when it is None this wrapper, not the library, allocates it with torch)."""
    M, K = A.dq4.shape[0], A.dq4.shape[1] * 2
    N = W.wq4.shape[0]
    if out is None:
        out = _buf(M * N * 2, torch.bfloat16, A.dq4.device)[: M * N].view(M, N)
    ca, cw = A.c_struct(), W.c_struct()
    _check(_lib.sq_gemm_static_scratch(ctypes.byref(fmt), ctypes.byref(ca), ctypes.byref(cw), _ptr(positions),
                                       M, N, K, _ptr(out), _ptr(acc_out), _stream(stream)), "sq_gemm_static_scratch")
    return out


def sq_gemm(fmt: sq_format, A: Encoded, W: Weights, positions: torch.Tensor | None = None,
            out: torch.Tensor | None = None, acc_out: torch.Tensor | None = None, stream=None,
            use_workspace: bool = True) -> torch.Tensor:
    """sq_gemm of the C ABI; decode-shaped calls (few rows) go through sq_gemm_ws with a scratch buffer
    cached per device (so calls on one device must not overlap on the GPU: keep them on one stream,
    or pass use_workspace=False)."""
    M, K = A.dq4.shape[0], A.dq4.shape[1] * 2
    N = W.wq4.shape[0]
    need = sq_gemm_workspace_bytes(fmt, M, N, K) if use_workspace else 0
    ws = _workspace(need, A.dq4.device) if need else None
    return sq_gemm_ws(fmt, A, W, positions, out=out, acc_out=acc_out, workspace=ws, stream=stream)


_workspaces: dict = {}


def _workspace(nbytes: int, device) -> torch.Tensor:
    key = str(device)
    buf = _workspaces.get(key)
    if buf is None or buf.numel() < nbytes:
        buf = torch.empty(max(nbytes, 1 << 20), dtype=torch.uint8, device=device)
        _workspaces[key] = buf
    return buf


def sq_decode(fmt: sq_format, A: Encoded, positions: torch.Tensor | None = None,
              out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    M, K = A.dq4.shape[0], A.dq4.shape[1] * 2
    if out is None:
        out = _buf(M * K * 2, torch.bfloat16, A.dq4.device)[: M * K].view(M, K)
    ca = A.c_struct()
    _check(_lib.sq_decode(ctypes.byref(fmt), ctypes.byref(ca), _ptr(positions), M, K, _ptr(out),
                          _stream(stream)), "sq_decode")
    return out


def sq_device_status(stream=None) -> int:
    return int(_lib.sq_device_status(_stream(stream)))


# ---------------------------------------------------------------------------- floating-point variant

@dataclass
class FpWeights:
    """Torch-owned buffers of the floating-point variant's weights."""
    wq4: torch.Tensor      # uint8 [N, K/2] E2M1 codes
    s_w: torch.Tensor      # float32 [N]
    w8: torch.Tensor       # uint8 [N, K] the same values as E4M3 bytes


def sq_fp_pack_weights(W: torch.Tensor, stream=None) -> FpWeights:
    N, K = _bf16_2d(W, "W")
    out = FpWeights(torch.empty(N, K // 2, dtype=torch.uint8, device=W.device),
                    torch.empty(max(N, 4), dtype=torch.float32, device=W.device)[:N],
                    torch.empty(N, K, dtype=torch.uint8, device=W.device))
    _check(_lib.sq_fp_pack_weights(_ptr(W), N, K, _ptr(out.wq4), _ptr(out.s_w), _ptr(out.w8), _stream(stream)),
           "sq_fp_pack_weights")
    return out


def sq_fp_encode(fmt: sq_format, X: torch.Tensor, positions: torch.Tensor | None = None, out: Encoded | None = None,
                 a8: torch.Tensor | None = None, stream=None):
    """Returns (Encoded, a8): the encoding (vals viewed as int8 holds E4M3 bytes) and the merged E4M3 operand."""
    M, K = _bf16_2d(X, "X")
    if out is None:
        out = alloc_encoded(fmt, M, K, X.device)
    if a8 is None:
        a8 = torch.empty(max(M * K, 16), dtype=torch.uint8, device=X.device)[: M * K].view(M, K)
    cs = out.c_struct()
    _check(_lib.sq_fp_encode(ctypes.byref(fmt), _ptr(X), M, K, _ptr(positions), ctypes.byref(cs), _ptr(a8),
                             _stream(stream)), "sq_fp_encode")
    return out, a8



def sq_fp_rmsnorm_encode(fmt: sq_format, X: torch.Tensor, gamma: torch.Tensor, eps: float, positions: torch.Tensor,
                         out: Encoded | None = None, a8: torch.Tensor | None = None, stream=None):
    """sq_fp_encode of rmsnorm(X) * gamma, the normalisation computed inside the encode; returns (Encoded, a8)."""
    M, K = _bf16_2d(X, "X")
    if gamma.dtype != torch.bfloat16 or gamma.numel() != K or not gamma.is_contiguous():
        raise ValueError("gamma must be a contiguous bf16 tensor of K elements")
    if out is None:
        out = alloc_encoded(fmt, M, K, X.device)
    if a8 is None:
        a8 = torch.empty(max(M * K, 16), dtype=torch.uint8, device=X.device)[: M * K].view(M, K)
    cs = out.c_struct()
    _check(_lib.sq_fp_rmsnorm_encode(ctypes.byref(fmt), _ptr(X), _ptr(gamma), ctypes.c_float(eps), M, K, _ptr(positions),
                                     ctypes.byref(cs), _ptr(a8), _stream(stream)), "sq_fp_rmsnorm_encode")
    return out, a8


def sq_fp_gemm(A: Encoded, a8: torch.Tensor, W: FpWeights, out: torch.Tensor | None = None,
               acc_out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    M, K = a8.shape
    N = W.w8.shape[0]
    if out is None:
        out = _buf(M * N * 2, torch.bfloat16, a8.device)[: M * N].view(M, N)
    _check(_lib.sq_fp_gemm(_ptr(A.s_hi), _ptr(a8), _ptr(W.s_w), _ptr(W.w8), M, N, K, _ptr(out), _ptr(acc_out),
                           _stream(stream)), "sq_fp_gemm")
    return out


def sq_fp_decode(fmt: sq_format, A: Encoded, positions: torch.Tensor | None = None, out: torch.Tensor | None = None,
                 stream=None) -> torch.Tensor:
    M, K = A.dq4.shape[0], A.dq4.shape[1] * 2
    if out is None:
        out = _buf(M * K * 2, torch.bfloat16, A.dq4.device)[: M * K].view(M, K)
    ca = A.c_struct()
    _check(_lib.sq_fp_decode(ctypes.byref(fmt), ctypes.byref(ca), _ptr(positions), M, K, _ptr(out), _stream(stream)),
           "sq_fp_decode")
    return out


# ---------------------------------------------------------------------------- SQ-format on weights

@dataclass
class SqWeights:
    """Torch-owned buffers of weights in SQ-format (implicit mask: the INT4 pattern 1000)."""
    wq4: torch.Tensor      # uint8 [N, K/2]
    w_hi: torch.Tensor     # int8 [N, K/b, k]
    s_high: torch.Tensor   # float32 [N]
    s_low: torch.Tensor    # float32 [N]


def sq_w_encode(fmt: sq_format, W: torch.Tensor, importance: torch.Tensor, stream=None) -> SqWeights:
    N, K = _bf16_2d(W, "W")
    if importance.dtype != torch.float32 or importance.shape != W.shape or not importance.is_contiguous():
        raise ValueError("importance must be a contiguous float32 tensor of W's shape")
    out = SqWeights(torch.empty(N, K // 2, dtype=torch.uint8, device=W.device),
                    torch.empty(N, K // fmt.bank, fmt.k, dtype=torch.int8, device=W.device),
                    torch.empty(max(N, 4), dtype=torch.float32, device=W.device)[:N],
                    torch.empty(max(N, 4), dtype=torch.float32, device=W.device)[:N])
    _check(_lib.sq_w_encode(ctypes.byref(fmt), _ptr(W), _ptr(importance), N, K, _ptr(out.wq4), _ptr(out.w_hi),
                            _ptr(out.s_high), _ptr(out.s_low), _stream(stream)), "sq_w_encode")
    return out


def sq_w_act_quant(X: torch.Tensor, stream=None):
    """Returns (xq int8 [M, K] in the product kernel's element order, s_x float32 [M])."""
    M, K = _bf16_2d(X, "X")
    xq = torch.empty(max(M * K, 16), dtype=torch.int8, device=X.device)[: M * K].view(M, K)
    s_x = torch.empty(max(M, 4), dtype=torch.float32, device=X.device)[:M]
    _check(_lib.sq_w_act_quant(_ptr(X), M, K, _ptr(xq), _ptr(s_x), _stream(stream)), "sq_w_act_quant")
    return xq, s_x


def sq_w_gemm(fmt: sq_format, xq: torch.Tensor, s_x: torch.Tensor, W: SqWeights, out: torch.Tensor | None = None,
              acc_out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    M, K = xq.shape
    N = W.wq4.shape[0]
    if out is None:
        out = _buf(M * N * 2, torch.bfloat16, xq.device)[: M * N].view(M, N)
    _check(_lib.sq_w_gemm(ctypes.byref(fmt), _ptr(xq), _ptr(s_x), _ptr(W.wq4), _ptr(W.w_hi), _ptr(W.s_high),
                          _ptr(W.s_low), M, N, K, _ptr(out), _ptr(acc_out), _stream(stream)), "sq_w_gemm")
    return out


def sq_probe_int8_tensor_rate(iterations: int, stream=None) -> float:
    """Launches the tensor-rate probe (tcgen05.mma.kind::i8 on resident operands, nothing else);
    returns the number of INT8 operations the launch issues.  Time it with CUDA events."""
    ops = ctypes.c_double(0.0)
    _check(_lib.sq_probe_int8_tensor_rate(int(iterations), ctypes.byref(ops), _stream(stream)), "sq_probe_int8_tensor_rate")
    return ops.value


def sq_probe_fp8_tensor_rate(iterations: int, stream=None) -> float:
    """The same probe for tcgen05.mma.kind::f8f6f4 (E4M3 x E4M3); returns the launch's floating-point operations."""
    ops = ctypes.c_double(0.0)
    _check(_lib.sq_probe_fp8_tensor_rate(int(iterations), ctypes.byref(ops), _stream(stream)), "sq_probe_fp8_tensor_rate")
    return ops.value


def sq_device_status_word() -> int:
    """Device address of the current device's status word."""
    out = ctypes.c_void_p(0)
    _check(_lib.sq_device_status_word(ctypes.byref(out)), "sq_device_status_word")
    return int(out.value)


def raw():
    """The ctypes CDLL itself (for tests that pass hand-made pointers)."""
    return _lib
