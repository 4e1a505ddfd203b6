"""Integer-only hash streams on torch int64 tensors.

Everything here is exact integer arithmetic (wrapping 64-bit multiply, logical
shifts emulated on signed int64), so the same call returns the same bits on a
CPU tensor and on a CUDA tensor.  Used only to generate inputs.
"""
from __future__ import annotations

import torch


def _s64(x: int) -> int:
    """Python int -> the signed 64-bit value with the same bit pattern."""
    x &= (1 << 64) - 1
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_M1 = _s64(0xBF58476D1CE4E5B9)
_M2 = _s64(0x94D049BB133111EB)


def lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of int64 bit patterns."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def splitmix64(x: torch.Tensor) -> torch.Tensor:
    """The splitmix64 output function (Steele, Lea, Flood 2014) on int64 bit patterns."""
    z = x + _GOLDEN
    z = (z ^ lsr(z, 30)) * _M1
    z = (z ^ lsr(z, 27)) * _M2
    return z ^ lsr(z, 31)


def stream_base(seed: int, stream: int) -> int:
    """A per-(seed, stream) 64-bit offset, computed with Python ints."""
    def sm(v):
        v = (v + 0x9E3779B97F4A7C15) & ((1 << 64) - 1)
        v = ((v ^ (v >> 30)) * 0xBF58476D1CE4E5B9) & ((1 << 64) - 1)
        v = ((v ^ (v >> 27)) * 0x94D049BB133111EB) & ((1 << 64) - 1)
        return v ^ (v >> 31)
    return _s64(sm(sm(seed & ((1 << 64) - 1)) ^ ((stream * 0xD6E8FEB86659FD93) & ((1 << 64) - 1))))


def hash_u64(seed: int, stream: int, idx: torch.Tensor) -> torch.Tensor:
    """64 pseudo-random bits per element of `idx` (int64), as int64 bit patterns."""
    return splitmix64(idx * _GOLDEN + stream_base(seed, stream))


def permutation(seed: int, stream: int, n: int, device="cpu") -> torch.Tensor:
    """A seeded permutation of [0, n): the argsort of distinct 64-bit hashes.

    splitmix64 is a bijection on 64-bit words and idx*odd + c is injective, so the
    hashes are distinct and the argsort does not depend on the sort's tie handling.
    """
    idx = torch.arange(n, dtype=torch.int64, device=device)
    return torch.argsort(hash_u64(seed, stream, idx))
