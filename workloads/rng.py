"""Counter-based seeded random numbers for the synthetic inputs.

Every value is a pure function of ``(seed, stream, index)``; nothing here holds
state, so the CPU checker and the GPU harness can each ask for the same slice of
the same stream on their own device and receive identical bits.  The generator
uses 64-bit integer arithmetic only (a SplitMix64-style finaliser over a Weyl
sequence), which ``torch`` evaluates identically on CPU and on CUDA.  Normal
deviates come from a 65 536-entry inverse-CDF table indexed by the top 16 random
bits, so no transcendental function is evaluated on either device.

This module is input generation only: it contains none of the arithmetic of the
verification step.
"""
from __future__ import annotations

import functools
import statistics

import torch

_GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_MASK64 = (1 << 64) - 1


def _s64(v: int) -> int:
    """Two's-complement view of an unsigned 64-bit constant."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def _mix_py(z: int) -> int:
    z &= _MASK64
    z = ((z ^ (z >> 30)) * _M1) & _MASK64
    z = ((z ^ (z >> 27)) * _M2) & _MASK64
    return z ^ (z >> 31)


def stream_key(seed: int, stream: int, *sub: int) -> int:
    """Derive the 64-bit base of a stream from a seed, a purpose id and sub-ids."""
    k = _mix_py(seed * _GOLDEN + 0x632BE59BD9B4E019)
    for s in (stream, *sub):
        k = _mix_py((k + (int(s) + 1) * _GOLDEN) & _MASK64)
    return k


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of an int64 tensor (torch's >> is arithmetic)."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def bits64(key: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """``count`` 64-bit words of stream ``key`` starting at element ``start`` (int64 bit patterns)."""
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    z = idx * _s64(_GOLDEN) + _s64(key)
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


def bits64_at(key: int, idx: torch.Tensor) -> torch.Tensor:
    """Same as :func:`bits64` for an arbitrary int64 index tensor."""
    z = idx.to(torch.int64) * _s64(_GOLDEN) + _s64(key)
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


@functools.lru_cache(maxsize=None)
def _normal_table_cpu() -> torch.Tensor:
    nd = statistics.NormalDist()
    vals = [nd.inv_cdf((k + 0.5) / 65536.0) for k in range(65536)]
    return torch.tensor(vals, dtype=torch.float64).to(torch.float32)


@functools.lru_cache(maxsize=None)
def _normal_table(device: str) -> torch.Tensor:
    return _normal_table_cpu().to(device)


def normal_f32(key: int, start: int, count: int, std: float, mean: float = 0.0,
               device="cpu") -> torch.Tensor:
    """fp32 deviates ``mean + std * z`` with ``z`` from the 16-bit inverse-CDF table."""
    b = bits64(key, start, count, device)
    z = _normal_table(str(device))[_lsr(b, 48)]
    out = z * torch.tensor(std, dtype=torch.float32, device=device)
    if mean != 0.0:
        out = out + torch.tensor(mean, dtype=torch.float32, device=device)
    return out


def normal_f32_at(key: int, idx: torch.Tensor, std: float) -> torch.Tensor:
    b = bits64_at(key, idx)
    z = _normal_table(str(idx.device))[_lsr(b, 48)]
    return z * torch.tensor(std, dtype=torch.float32, device=idx.device)


def uniform01(key: int, start: int, count: int) -> torch.Tensor:
    """fp64 uniforms in [0, 1) on the CPU (53 random bits each)."""
    return _lsr(bits64(key, start, count), 11).to(torch.float64) / float(1 << 53)


def randint(key: int, start: int, count: int, lo: int, hi: int, device="cpu") -> torch.Tensor:
    """Integers uniform on the inclusive range [lo, hi] (int64)."""
    span = hi - lo + 1
    return _lsr(bits64(key, start, count, device), 1) % span + lo


def permutation(key: int, n: int) -> torch.Tensor:
    """A seeded permutation of range(n): argsort of n random words (ties by index)."""
    b = _lsr(bits64(key, 0, n), 1)
    return torch.sort(b, stable=True).indices
