"""Counter-based random numbers: element `index` of stream (`seed`, `tensor_id`).

Every value is a pure function of (seed, tensor_id, index), so any slice of any
tensor can be produced in any order, on the host or on a GPU, with the same
integers.  The mixer is splitmix64 (Steele, Lea, Flood 2014; the finaliser of
Java's SplittableRandom), evaluated in wrapping 64-bit integer arithmetic.
"""
from __future__ import annotations

import torch

_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB


def _s64(x: int) -> int:
    """Reinterpret an unsigned 64-bit integer as the signed value torch stores."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def splitmix64_scalar(x: int) -> int:
    """splitmix64 output for the 64-bit state `x` (plain Python integers)."""
    z = (x + _GOLDEN) & _M64
    z = ((z ^ (z >> 30)) * _C1) & _M64
    z = ((z ^ (z >> 27)) * _C2) & _M64
    return z ^ (z >> 31)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of int64 data (torch's >> is arithmetic)."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def _mix(z: torch.Tensor) -> torch.Tensor:
    z = z + _s64(_GOLDEN)
    z = (z ^ _lsr(z, 30)) * _s64(_C1)
    z = (z ^ _lsr(z, 27)) * _s64(_C2)
    return z ^ _lsr(z, 31)


def stream_base(seed: int, tensor_id: int) -> int:
    """64-bit base of stream (seed, tensor_id)."""
    return splitmix64_scalar(splitmix64_scalar(seed & _M64) ^ ((tensor_id * 0xD1342543DE82EF95) & _M64))


def hash_u64(seed: int, tensor_id: int, index: torch.Tensor) -> torch.Tensor:
    """64 random bits per element of `index` (int64 tensor), as int64 bit patterns."""
    base = stream_base(seed, tensor_id)
    return _mix(index * _s64(_GOLDEN) + _s64(base))


def uniform01(bits: torch.Tensor) -> torch.Tensor:
    """Map 64-bit patterns to float64 in the open interval (0, 1): (top 53 bits + 0.5) / 2^53."""
    return (_lsr(bits, 11).to(torch.float64) + 0.5) * (1.0 / (1 << 53))
