"""Counter-based random numbers for the synthetic inputs.

Every draw is a pure function of (seed, stream, counter), so any element can be
regenerated anywhere and the same arrays come out on the CPU and on a GPU.
All arithmetic is wrapping 64-bit integer arithmetic on torch int64 tensors;
no floating-point reduction is involved, so results do not depend on the device.

This module holds no tensor-algebra arithmetic: it only makes inputs.
"""
from __future__ import annotations

import torch

_MASK64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Two's-complement reinterpretation of an unsigned 64-bit constant."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_M1 = _s64(0xBF58476D1CE4E5B9)
_M2 = _s64(0x94D049BB133111EB)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of int64 lanes (torch's >> is arithmetic)."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def _mix(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def _mix_int(z: int) -> int:
    z &= _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


def stream_key(seed: int, stream: int) -> int:
    """One 64-bit key per (seed, stream); distinct streams are decorrelated by two mixes."""
    return _mix_int(_mix_int(seed * 0x9E3779B97F4A7C15 + 0x1234567) ^ (stream * 0xD1B54A32D192ED03))


def bits64(seed: int, stream: int, counter: torch.Tensor) -> torch.Tensor:
    """64 random bits (as int64) for each int64 counter value."""
    key = _s64(stream_key(seed, stream))
    return _mix(counter * _GOLDEN + key)


def counters(n: int, device, offset: int = 0) -> torch.Tensor:
    return torch.arange(offset, offset + n, dtype=torch.int64, device=device)


def uniform(seed: int, stream: int, n: int, device="cpu", offset: int = 0) -> torch.Tensor:
    """n doubles in [0, 1) with 53 random bits each."""
    b = bits64(seed, stream, counters(n, device, offset))
    return _lsr(b, 11).to(torch.float64) * (1.0 / 9007199254740992.0)


def uniform_at(seed: int, stream: int, counter: torch.Tensor) -> torch.Tensor:
    return _lsr(bits64(seed, stream, counter), 11).to(torch.float64) * (1.0 / 9007199254740992.0)


def below(seed: int, stream: int, n: int, bound: int, device="cpu", offset: int = 0) -> torch.Tensor:
    """n int64 values uniform in [0, bound) (floor of u * bound; bound < 2**52)."""
    u = uniform(seed, stream, n, device, offset)
    return torch.clamp((u * float(bound)).to(torch.int64), max=bound - 1)


def below_at(seed: int, stream: int, counter: torch.Tensor, bound: int) -> torch.Tensor:
    u = uniform_at(seed, stream, counter)
    return torch.clamp((u * float(bound)).to(torch.int64), max=bound - 1)


def symmetric(seed: int, stream: int, n: int, device="cpu", offset: int = 0) -> torch.Tensor:
    """n doubles in [-1, 1): 2u - 1."""
    return uniform(seed, stream, n, device, offset) * 2.0 - 1.0


def permutation(seed: int, stream: int, n: int, device="cpu") -> torch.Tensor:
    """A seeded permutation of 0..n-1: rank the counters by their hash (ties broken by index)."""
    b = bits64(seed, stream, counters(n, device))
    # stable sort on the hash; a 64-bit collision is harmless (still a permutation)
    return torch.sort(b, stable=True).indices
