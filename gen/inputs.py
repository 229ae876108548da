"""Seeded synthetic inputs for the SQ-format hot path.

This module only draws numbers; it holds none of the method's arithmetic (no
quantisation, no selection, no packing) so that both the CPU oracle's tests and
the CUDA path's tests can be fed from it without sharing any of the method.

Every value is a pure function of (seed, stream, element index): a splitmix64
hash of a counter gives 64 uniform bits, two of them give one Box-Muller normal
in fp64, and the final cast to bf16 is round-to-nearest-even.  The same code runs
on the CPU and on a CUDA device (torch integer/fp64 ops); a tensor produced on a
device and then copied to the host is the input both sides see, so nothing
depends on the two devices' libm agreeing bit for bit.

The tensors stand in for the activations, weights and calibration batches of the
decoder linear layers the paper evaluates (Section 4.1): heavy-tailed values
(Student-t, nu = 3, or N(0,1)), a small fixed set of outlier channels scaled by a
large factor in both the calibration batch and the test batch, and N(0, 0.02^2)
weights.
"""
from __future__ import annotations

import math

import torch

# stream ids (added to the seed before hashing)
STREAM_ACT = 0
STREAM_WEIGHT = 1
STREAM_CALIB = 2
STREAM_OUTLIER = 3

_MASK64 = (1 << 64) - 1


def _s64(v: int) -> int:
    """Two's-complement reinterpretation of a 64-bit pattern as a Python int."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_C1 = _s64(0xBF58476D1CE4E5B9)
_C2 = _s64(0x94D049BB133111EB)


def _lshr(x: torch.Tensor, s: int) -> torch.Tensor:
    return (x >> s) & ((1 << (64 - s)) - 1)


def _splitmix64(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on int64 tensors holding 64-bit patterns (wrapping)."""
    z = x + _GOLDEN
    z = (z ^ _lshr(z, 30)) * _C1
    z = (z ^ _lshr(z, 27)) * _C2
    return z ^ _lshr(z, 31)


def _key(seed: int, stream: int, lane: int) -> int:
    """A 64-bit key per (seed, stream, lane) so that streams never overlap."""
    k = (seed * 0x100000001B3 + stream * 0x9E3779B1 + lane * 0x85EBCA6B + 0x243F6A8885A308D3) & _MASK64
    # one scalar splitmix round in Python ints
    z = (k + 0x9E3779B97F4A7C15) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return _s64(z ^ (z >> 31))


def _uniform(counter: torch.Tensor, key: int) -> torch.Tensor:
    """fp64 uniforms in (0, 1) from a counter tensor and a key."""
    bits = _splitmix64(counter ^ key)
    return (_lshr(bits, 11).to(torch.float64) + 0.5) * (1.0 / 9007199254740992.0)


def _normal(first: int, count: int, seed: int, stream: int, lane: int, device) -> torch.Tensor:
    """`count` standard normals (fp64) for element indices first .. first+count-1."""
    idx = torch.arange(first, first + count, dtype=torch.int64, device=device)
    u1 = _uniform(idx * 2, _key(seed, stream, lane))
    u2 = _uniform(idx * 2 + 1, _key(seed, stream, lane))
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def outlier_channels(K: int, fraction: float, seed: int) -> torch.Tensor:
    """A fixed, seeded set of floor(fraction*K) distinct channel indices (sorted, CPU int64)."""
    n = int(math.floor(fraction * K))
    if n <= 0:
        return torch.empty(0, dtype=torch.int64)
    j = torch.arange(K, dtype=torch.int64)
    score = _splitmix64(j ^ _key(seed, STREAM_OUTLIER, 0))
    order = torch.argsort(score, stable=True)
    return torch.sort(order[:n]).values


def _values(rows: int, cols: int, seed: int, stream: int, dist: str, device, row0: int = 0) -> torch.Tensor:
    first, count = row0 * cols, rows * cols
    z0 = _normal(first, count, seed, stream, 0, device)
    if dist == "normal":
        v = z0
    elif dist == "student_t3":
        z1 = _normal(first, count, seed, stream, 1, device)
        z2 = _normal(first, count, seed, stream, 2, device)
        z3 = _normal(first, count, seed, stream, 3, device)
        v = z0 / torch.sqrt((z1 * z1 + z2 * z2 + z3 * z3) / 3.0)
    else:
        raise ValueError(f"unknown distribution {dist!r}")
    return v.view(rows, cols)


def activations(M: int, K: int, *, seed: int = 0, dist: str = "student_t3",
                outlier_fraction: float = 0.01, outlier_scale: float = 20.0,
                stream: int = STREAM_ACT, device="cpu", chunk_rows: int = 1024) -> torch.Tensor:
    """bf16 [M, K] activations: `dist` values with a fixed set of channels scaled up.

    The outlier channel set depends on (K, outlier_fraction, seed) only, so a
    calibration batch (stream=STREAM_CALIB) and a test batch share it.
    """
    out = torch.empty(M, K, dtype=torch.bfloat16, device=device)
    ch = outlier_channels(K, outlier_fraction, seed).to(device)
    for r0 in range(0, M, chunk_rows):
        r = min(chunk_rows, M - r0)
        v = _values(r, K, seed, stream, dist, device, row0=r0)
        if ch.numel():
            v[:, ch] *= outlier_scale
        out[r0:r0 + r] = v.to(torch.float32).to(torch.bfloat16)
    return out


def calibration_batch(T: int, K: int, **kw) -> torch.Tensor:
    """bf16 [T, K] calibration activations (same outlier channels as `activations`)."""
    kw.setdefault("stream", STREAM_CALIB)
    return activations(T, K, **kw)


def weights(N: int, K: int, *, seed: int = 0, std: float = 0.02, device="cpu",
            chunk_rows: int = 1024) -> torch.Tensor:
    """bf16 [N, K] weights ~ N(0, std^2), K contiguous."""
    out = torch.empty(N, K, dtype=torch.bfloat16, device=device)
    for r0 in range(0, N, chunk_rows):
        r = min(chunk_rows, N - r0)
        v = _values(r, K, seed, STREAM_WEIGHT, "normal", device, row0=r0) * std
        out[r0:r0 + r] = v.to(torch.float32).to(torch.bfloat16)
    return out


def bf16_bits(t: torch.Tensor):
    """uint16 numpy view of a bf16 tensor's bits (copied to the host if needed)."""
    import numpy as np
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def from_bf16_bits(a, device="cpu") -> torch.Tensor:
    """bf16 tensor from a uint16 numpy array of bf16 bit patterns."""
    import numpy as np
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(device)
