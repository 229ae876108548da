"""ctypes front end of the CPU oracle (`sq_oracle.cpp`).  TEST INFRASTRUCTURE ONLY.

Only the test suite, the smoke check and the benchmark's CPU-baseline leg may
import this package; the CUDA library and its Python binding never do.  All
arrays are numpy; bf16 tensors travel as uint16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sq_oracle.cpp")
_SRC_FP = os.path.join(_HERE, "sq_oracle_fp.cpp")
_SRC_W = os.path.join(_HERE, "sq_oracle_w.cpp")
_LIB = os.path.join(_HERE, "libsq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2, no fast-math, OpenMP over rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_SRC_FP), os.path.getmtime(_SRC_W)):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC",
                               "-o", tmp, _SRC, _SRC_FP, _SRC_W])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.sqo_equivalent_bits.restype = ctypes.c_double
        _lib.sqo_equivalent_bits.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_int]
        _lib.sqo_num_threads.restype = ctypes.c_int
        _lib.sqo_gemm.restype = ctypes.c_int
        _lib.sqo_gemm_indep.restype = ctypes.c_int
    return _lib


def _p(a):
    if a is None:
        return ctypes.c_void_p(0)
    assert a.flags["C_CONTIGUOUS"]
    return ctypes.c_void_p(a.ctypes.data)


def _l(v):
    return ctypes.c_long(int(v))


def num_threads() -> int:
    return int(_load().sqo_num_threads())


def equivalent_bits(h_high: float, h_low: float, s: float, on_weights: bool) -> float:
    return float(_load().sqo_equivalent_bits(h_high, h_low, s, int(on_weights)))


@dataclass
class Encoded:
    dq4: np.ndarray      # uint8 [M, K/2]
    vals: np.ndarray     # int8  [M, G, k]
    idx: np.ndarray | None  # uint8 [M, G, k]; None for static positions
    s_hi: np.ndarray     # float32 [M]
    s_lo: np.ndarray     # float32 [M]
    shift: np.ndarray    # uint8 [M]


@dataclass
class Weights:
    wq4: np.ndarray      # uint8 [N, K/2]
    s_w: np.ndarray      # float32 [N]
    colsum: np.ndarray   # int32 [N]
    w_sparse: np.ndarray | None  # int8 [N, G*k]; None for dynamic positions
    wq: np.ndarray       # int8 [N, K] unpacked codes (convenience for tests)


def calib_positions(b: int, k: int, calib_bits: np.ndarray, W_bits: np.ndarray | None = None,
                    return_importance: bool = False):
    T, K = calib_bits.shape
    assert K % b == 0 and calib_bits.dtype == np.uint16
    N = 0 if W_bits is None else W_bits.shape[0]
    pos = np.zeros((K // b, k), dtype=np.uint8)
    imp = np.zeros(K, dtype=np.float64) if return_importance else None
    _load().sqo_calib_positions(ctypes.c_int(b), ctypes.c_int(k), _p(calib_bits), _l(T), _l(K),
                                _p(W_bits), _l(N), _p(pos), _p(imp))
    return (pos, imp) if return_importance else pos


def pack_weights(b: int, k: int, W_bits: np.ndarray, positions: np.ndarray | None = None) -> Weights:
    N, K = W_bits.shape
    assert K % b == 0 and K % 2 == 0 and W_bits.dtype == np.uint16
    G = K // b
    wq4 = np.zeros((N, K // 2), dtype=np.uint8)
    s_w = np.zeros(N, dtype=np.float32)
    colsum = np.zeros(N, dtype=np.int32)
    w_sparse = np.zeros((N, G * k), dtype=np.int8) if positions is not None else None
    wq = np.zeros((N, K), dtype=np.int8)
    _load().sqo_pack_weights(ctypes.c_int(b), ctypes.c_int(k), _p(W_bits), _l(N), _l(K), _p(positions),
                             _p(wq4), _p(s_w), _p(colsum), _p(w_sparse), _p(wq))
    return Weights(wq4, s_w, colsum, w_sparse, wq)


def encode(b: int, k: int, X_bits: np.ndarray, positions: np.ndarray | None = None) -> Encoded:
    M, K = X_bits.shape
    assert K % b == 0 and K % 2 == 0 and X_bits.dtype == np.uint16
    G = K // b
    dq4 = np.zeros((M, K // 2), dtype=np.uint8)
    vals = np.zeros((M, G, k), dtype=np.int8)
    idx = np.zeros((M, G, k), dtype=np.uint8) if positions is None else None
    s_hi = np.zeros(M, dtype=np.float32)
    s_lo = np.zeros(M, dtype=np.float32)
    shift = np.zeros(M, dtype=np.uint8)
    _load().sqo_encode(ctypes.c_int(b), ctypes.c_int(k), _p(X_bits), _l(M), _l(K), _p(positions),
                       _p(dq4), _p(vals), _p(idx), _p(s_hi), _p(s_lo), _p(shift))
    return Encoded(dq4, vals, idx, s_hi, s_lo, shift)


def gemm(b: int, k: int, A: Encoded, W: Weights, positions: np.ndarray | None = None,
         rows=None, cols=None):
    """Returns (acc int32, ref32 float32, out bf16-bits uint16), each [n_rows, n_cols]."""
    M, Kh = A.dq4.shape
    K = Kh * 2
    N = W.wq4.shape[0]
    rows_a = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    cols_a = None if cols is None else np.ascontiguousarray(cols, dtype=np.int64)
    R = M if rows_a is None else len(rows_a)
    C = N if cols_a is None else len(cols_a)
    acc = np.zeros((R, C), dtype=np.int32)
    ref = np.zeros((R, C), dtype=np.float32)
    out = np.zeros((R, C), dtype=np.uint16)
    ov = _load().sqo_gemm(ctypes.c_int(b), ctypes.c_int(k), _p(A.dq4), _p(A.vals), _p(A.idx),
                          _p(positions), _p(A.s_hi), _p(A.shift), _p(W.wq4), _p(W.s_w),
                          _l(M), _l(N), _l(K), _p(rows_a), _l(R), _p(cols_a), _l(C),
                          _p(acc), _p(ref), _p(out))
    if ov:
        raise OverflowError("an accumulator does not fit in int32")
    return acc, ref, out


def decode(b: int, k: int, A: Encoded, positions: np.ndarray | None = None):
    """Returns (x_hat float32 [M,K], x_hat bf16-bits uint16 [M,K])."""
    M, Kh = A.dq4.shape
    K = Kh * 2
    xf = np.zeros((M, K), dtype=np.float32)
    xb = np.zeros((M, K), dtype=np.uint16)
    _load().sqo_decode(ctypes.c_int(b), ctypes.c_int(k), _p(A.dq4), _p(A.vals), _p(A.idx), _p(positions),
                       _p(A.s_hi), _p(A.s_lo), _l(M), _l(K), _p(xf), _p(xb))
    return xf, xb


def encode_indep(b: int, k: int, X_bits: np.ndarray, positions: np.ndarray) -> Encoded:
    """Static positions with independent scales of the two parts (s_lo is not tied to s_hi; shift = 0)."""
    M, K = X_bits.shape
    assert K % b == 0 and K % 2 == 0 and X_bits.dtype == np.uint16 and positions is not None
    G = K // b
    dq4 = np.zeros((M, K // 2), dtype=np.uint8)
    vals = np.zeros((M, G, k), dtype=np.int8)
    s_hi = np.zeros(M, dtype=np.float32)
    s_lo = np.zeros(M, dtype=np.float32)
    shift = np.zeros(M, dtype=np.uint8)
    _load().sqo_encode_indep(ctypes.c_int(b), ctypes.c_int(k), _p(X_bits), _l(M), _l(K), _p(positions),
                             _p(dq4), _p(vals), _p(s_hi), _p(s_lo), _p(shift))
    return Encoded(dq4, vals, None, s_hi, s_lo, shift)


def gemm_indep(b: int, k: int, A: Encoded, W: Weights, positions: np.ndarray, rows=None, cols=None):
    """Returns (acc_lo int32, acc_hi int32, ref32 float32, out bf16-bits uint16), each [n_rows, n_cols]."""
    M, Kh = A.dq4.shape
    K = Kh * 2
    N = W.wq4.shape[0]
    rows_a = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    cols_a = None if cols is None else np.ascontiguousarray(cols, dtype=np.int64)
    R = M if rows_a is None else len(rows_a)
    C = N if cols_a is None else len(cols_a)
    lo = np.zeros((R, C), dtype=np.int32)
    hi = np.zeros((R, C), dtype=np.int32)
    ref = np.zeros((R, C), dtype=np.float32)
    out = np.zeros((R, C), dtype=np.uint16)
    ov = _load().sqo_gemm_indep(ctypes.c_int(b), ctypes.c_int(k), _p(A.dq4), _p(A.vals), _p(positions),
                                _p(A.s_hi), _p(A.s_lo), _p(W.wq4), _p(W.s_w), _l(M), _l(N), _l(K),
                                _p(rows_a), _l(R), _p(cols_a), _l(C), _p(lo), _p(hi), _p(ref), _p(out))
    if ov:
        raise OverflowError("an accumulator does not fit in int32")
    return lo, hi, ref, out


# ---------------------------------------------------------------------------- floating-point variant (FP8 sparse + FP4 dense)

@dataclass
class FpEncoded:
    dq4: np.ndarray      # uint8 [M, K/2] E2M1 codes, two per byte
    vals: np.ndarray     # uint8 [M, G, k] E4M3 codes
    idx: np.ndarray | None
    s_hi: np.ndarray
    s_lo: np.ndarray
    shift: np.ndarray
    a8: np.ndarray       # uint8 [M, K] merged E4M3 operand


@dataclass
class FpWeights:
    wq4: np.ndarray      # uint8 [N, K/2] E2M1 codes
    s_w: np.ndarray
    w8: np.ndarray       # uint8 [N, K] the same values as E4M3 codes


def fp_tables():
    e2 = np.zeros(16, dtype=np.float64)
    e4 = np.zeros(256, dtype=np.float64)
    _load().sqo_fp_tables(_p(e2), _p(e4))
    return e2, e4


def fp_round(kind: str, values: np.ndarray) -> np.ndarray:
    v = np.ascontiguousarray(values, dtype=np.float64).ravel()
    out = np.zeros(v.size, dtype=np.uint8)
    _load().sqo_fp_round(ctypes.c_int(0 if kind == "e2m1" else 1), _p(v), _l(v.size), _p(out))
    return out.reshape(np.shape(values))


def fp_pack_weights(W_bits: np.ndarray) -> FpWeights:
    N, K = W_bits.shape
    wq4 = np.zeros((N, K // 2), dtype=np.uint8)
    s_w = np.zeros(N, dtype=np.float32)
    w8 = np.zeros((N, K), dtype=np.uint8)
    _load().sqo_fp_pack_weights(_p(W_bits), _l(N), _l(K), _p(wq4), _p(s_w), _p(w8))
    return FpWeights(wq4, s_w, w8)


def fp_encode(b: int, k: int, X_bits: np.ndarray, positions: np.ndarray | None = None) -> FpEncoded:
    M, K = X_bits.shape
    G = K // b
    dq4 = np.zeros((M, K // 2), dtype=np.uint8)
    vals = np.zeros((M, G, k), dtype=np.uint8)
    idx = np.zeros((M, G, k), dtype=np.uint8) if positions is None else None
    s_hi = np.zeros(M, dtype=np.float32)
    s_lo = np.zeros(M, dtype=np.float32)
    shift = np.zeros(M, dtype=np.uint8)
    a8 = np.zeros((M, K), dtype=np.uint8)
    _load().sqo_fp_encode(ctypes.c_int(b), ctypes.c_int(k), _p(X_bits), _l(M), _l(K), _p(positions), _p(dq4), _p(vals),
                          _p(idx), _p(s_hi), _p(s_lo), _p(shift), _p(a8))
    return FpEncoded(dq4, vals, idx, s_hi, s_lo, shift, a8)


def fp_gemm(A: FpEncoded, W: FpWeights, rows=None, cols=None):
    """Returns (acc float32, sum of |products| float32, ref32 float32, out bf16-bits), each [n_rows, n_cols]."""
    M, K = A.a8.shape
    N = W.wq4.shape[0]
    rows_a = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    cols_a = None if cols is None else np.ascontiguousarray(cols, dtype=np.int64)
    R = M if rows_a is None else len(rows_a)
    C = N if cols_a is None else len(cols_a)
    acc = np.zeros((R, C), dtype=np.float32)
    sabs = np.zeros((R, C), dtype=np.float32)
    ref = np.zeros((R, C), dtype=np.float32)
    out = np.zeros((R, C), dtype=np.uint16)
    _load().sqo_fp_gemm(_p(A.a8), _p(A.s_hi), _p(W.wq4), _p(W.s_w), _l(M), _l(N), _l(K), _p(rows_a), _l(R), _p(cols_a),
                        _l(C), _p(acc), _p(sabs), _p(ref), _p(out))
    return acc, sabs, ref, out


def fp_decode(b: int, k: int, A: FpEncoded, positions: np.ndarray | None = None):
    M, K = A.a8.shape
    xf = np.zeros((M, K), dtype=np.float32)
    xb = np.zeros((M, K), dtype=np.uint16)
    _load().sqo_fp_decode(ctypes.c_int(b), ctypes.c_int(k), _p(A.dq4), _p(A.vals), _p(A.idx), _p(positions), _p(A.s_hi),
                          _p(A.s_lo), _l(M), _l(K), _p(xf), _p(xb))
    return xf, xb


# ---------------------------------------------------------------------------- SQ-format on weights (Algorithm 1's format)

@dataclass
class SqWeights:
    wq4: np.ndarray      # uint8 [N, K/2]: INT4 codes, the pattern 1000 at high-precision places
    w_hi: np.ndarray     # int8 [N, G, k]: the high-precision values, in position order
    s_high: np.ndarray   # float32 [N]
    s_low: np.ndarray    # float32 [N]


def w_encode(b: int, k: int, W_bits: np.ndarray, importance: np.ndarray) -> SqWeights:
    N, K = W_bits.shape
    imp = np.ascontiguousarray(importance, dtype=np.float32)
    wq4 = np.zeros((N, K // 2), dtype=np.uint8)
    w_hi = np.zeros((N, K // b, k), dtype=np.int8)
    s_high = np.zeros(N, dtype=np.float32)
    s_low = np.zeros(N, dtype=np.float32)
    _load().sqo_w_encode(ctypes.c_int(b), ctypes.c_int(k), _p(W_bits), _p(imp), _l(N), _l(K), _p(wq4), _p(w_hi),
                         _p(s_high), _p(s_low))
    return SqWeights(wq4, w_hi, s_high, s_low)


def w_decode(b: int, k: int, Wq: SqWeights) -> np.ndarray:
    N, Kh = Wq.wq4.shape
    out = np.zeros((N, Kh * 2), dtype=np.float32)
    _load().sqo_w_decode(ctypes.c_int(b), ctypes.c_int(k), _p(Wq.wq4), _p(Wq.w_hi), _p(Wq.s_high), _p(Wq.s_low), _l(N),
                         _l(Kh * 2), _p(out))
    return out


def act_quant8(X_bits: np.ndarray):
    M, K = X_bits.shape
    xq = np.zeros((M, K), dtype=np.int8)
    s_x = np.zeros(M, dtype=np.float32)
    _load().sqo_act_quant8(_p(X_bits), _l(M), _l(K), _p(xq), _p(s_x))
    return xq, s_x


def w_gemm(b: int, k: int, xq: np.ndarray, s_x: np.ndarray, Wq: SqWeights):
    """Returns (acc_lo int32, acc_hi int32, ref32 float32, out bf16-bits), each [M, N]."""
    M, K = xq.shape
    N = Wq.wq4.shape[0]
    lo = np.zeros((M, N), dtype=np.int32)
    hi = np.zeros((M, N), dtype=np.int32)
    ref = np.zeros((M, N), dtype=np.float32)
    out = np.zeros((M, N), dtype=np.uint16)
    _load().sqo_w_gemm(ctypes.c_int(b), ctypes.c_int(k), _p(xq), _p(s_x), _p(Wq.wq4), _p(Wq.w_hi), _p(Wq.s_high),
                       _p(Wq.s_low), _l(M), _l(N), _l(K), _p(lo), _p(hi), _p(ref), _p(out))
    return lo, hi, ref, out


# ---------------------------------------------------------------------------- the producer of an activation
#
# The decoder layers whose prefill the appendix "End-to-End Latency Analysis" times feed two of
# their four quantised linears from a root-mean-square layer normalisation (y = x / rms(x) * gamma).
# The paper does not spell the normalisation out; this is its usual definition with the roundings
# of a bf16 decoder made explicit (the reading the CUDA path is held to):
#   ms = (sum_j x_j^2) / K            in fp64 (every square of a bf16 value is exact there)
#   r  = fp32(1 / sqrt(ms + eps))     one rounding to fp32
#   t  = bf16(fp32(x) * r)            fp32 product, round-to-nearest-even to bf16
#   y  = bf16(fp32(t) * fp32(gamma))  the product of two bf16 values is exact in fp32; one rounding
# A row is "ambiguous" when 1/sqrt(ms + eps) lies so close to the middle between two fp32 values
# that the order of the fp64 additions could decide r; callers assert there is none.

def _bf16_rne_bits(f32: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(f32, dtype=np.float32).view(np.uint32).astype(np.uint64)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


def rmsnorm(X_bits: np.ndarray, gamma_bits: np.ndarray, eps: float):
    """(y bits uint16 [M,K], r float32 [M], ambiguous bool [M]) of the definition above."""
    assert X_bits.dtype == np.uint16 and gamma_bits.dtype == np.uint16 and gamma_bits.shape == (X_bits.shape[1],)
    M, K = X_bits.shape
    x32 = (X_bits.astype(np.uint32) << 16).view(np.float32)
    g32 = (gamma_bits.astype(np.uint32) << 16).view(np.float32)
    x64 = x32.astype(np.float64)
    ms = np.array([float(np.sum(x64[m] * x64[m])) for m in range(M)], dtype=np.float64) / float(K)
    r64 = 1.0 / np.sqrt(ms + float(np.float32(eps)))
    r = r64.astype(np.float32)
    # distance of r64 from the nearest rounding boundary of fp32, in units of the fp32 spacing
    up = np.nextafter(r, np.float32(np.inf)).astype(np.float64)
    dn = np.nextafter(r, np.float32(-np.inf)).astype(np.float64)
    r_d = r.astype(np.float64)
    with np.errstate(invalid="ignore", divide="ignore"):
        d_up = np.abs(r64 - (r_d + up) / 2) / (up - r_d)
        d_dn = np.abs(r64 - (r_d + dn) / 2) / (r_d - dn)
    ambiguous = np.minimum(d_up, d_dn) < 1e-9
    t = _bf16_rne_bits(x32 * r[:, None])
    t32 = (t.astype(np.uint32) << 16).view(np.float32)
    y = _bf16_rne_bits(t32 * g32[None, :])
    return y, r, ambiguous


def rmsnorm_encode(b: int, k: int, X_bits: np.ndarray, gamma_bits: np.ndarray, eps: float, positions: np.ndarray):
    """The normalisation followed by the static-position encode of its output (Algorithm 2)."""
    y, _, ambiguous = rmsnorm(X_bits, gamma_bits, eps)
    assert not ambiguous.any()
    return encode(b, k, y, positions), y
