"""Small numpy helpers owned by the tests (independent of both implementations)."""
from fractions import Fraction

import numpy as np
import torch


def bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def unpack_nibbles(packed: np.ndarray) -> np.ndarray:
    """uint8 [..., K/2] -> int8 [..., K]; low nibble first, two's complement."""
    lo = (packed & 0xF).astype(np.int16)
    hi = (packed >> 4).astype(np.int16)
    lo = np.where(lo >= 8, lo - 16, lo)
    hi = np.where(hi >= 8, hi - 16, hi)
    out = np.stack([lo, hi], axis=-1).reshape(*packed.shape[:-1], packed.shape[-1] * 2)
    return out.astype(np.int8)


def rne_fraction(p: Fraction) -> int:
    """Round-half-to-even of an exact rational."""
    fl = p.numerator // p.denominator
    rem = p - fl
    if rem > Fraction(1, 2):
        return fl + 1
    if rem < Fraction(1, 2):
        return fl
    return fl if fl % 2 == 0 else fl + 1


def sparse_dense_split(enc, b, k, positions=None):
    """(q_lo int64 [M,K], q_hi int64 [M,K] zero off-support, support bool [M,K]) from an encoding."""
    q_lo = unpack_nibbles(enc.dq4).astype(np.int64)
    M, K = q_lo.shape
    G = K // b
    idx = enc.idx if enc.idx is not None else np.broadcast_to(positions[None], (M, G, k))
    cols = (np.arange(G)[None, :, None] * b + idx.astype(np.int64)).reshape(M, G * k)
    q_hi = np.zeros((M, K), dtype=np.int64)
    sup = np.zeros((M, K), dtype=bool)
    rows = np.repeat(np.arange(M), G * k).reshape(M, G * k)
    q_hi[rows, cols] = enc.vals.reshape(M, G * k).astype(np.int64)
    sup[rows, cols] = True
    return q_lo, q_hi, sup
