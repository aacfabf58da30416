"""Seeded, counter-based synthetic tensors (inputs only; none of the MoE arithmetic lives here).

Every element is a pure function of (seed, element index), so a tensor can be
generated in chunks, on the CPU or on a CUDA device, and come out the same up
to the last-ulp behaviour of the device's fp64 log/cos/sin (which, after the
final rounding to fp32/bf16, is almost never visible).  Consumers that must see
identical bits on both sides copy ONE generated tensor to where it is needed;
they never generate it twice on different devices.

Generator: splitmix64 finaliser over a 64-bit counter -> two 53-bit uniforms ->
Box-Muller -> N(0,1) in fp64 -> scale -> fp32 -> (round to nearest even) bf16.
"""
from __future__ import annotations

import math

import torch

_GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_MASK64 = (1 << 64) - 1


def _s64(v: int) -> int:
    """Reinterpret an unsigned 64-bit integer as the signed value torch.int64 holds."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def _lsr(z: torch.Tensor, n: int) -> torch.Tensor:
    """Logical right shift on int64 (torch's >> is arithmetic)."""
    return (z >> n) & ((1 << (64 - n)) - 1)


def _mix(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


def hash_u64(seed: int, idx: torch.Tensor) -> torch.Tensor:
    """splitmix64 output number idx of the stream started at `seed` (int64 bit patterns)."""
    start = _s64(_mix_int(seed))
    return _mix(idx * _s64(_GOLDEN) + start)


def _mix_int(v: int) -> int:
    v = (v + _GOLDEN) & _MASK64
    v = ((v ^ (v >> 30)) * _M1) & _MASK64
    v = ((v ^ (v >> 27)) * _M2) & _MASK64
    return v ^ (v >> 31)


def uniform01(seed: int, idx: torch.Tensor) -> torch.Tensor:
    """fp64 uniforms in (0,1), 53 random bits each, never exactly 0 or 1."""
    bits = _lsr(hash_u64(seed, idx), 11)
    return (bits.to(torch.float64) + 0.5) * (1.0 / (1 << 53))


def normal(seed: int, shape, std: float = 1.0, dtype=torch.float32, device="cpu",
           chunk: int = 1 << 24) -> torch.Tensor:
    """N(0, std^2) tensor of `shape`; element i uses counters 2*(i//2) and 2*(i//2)+1."""
    n = 1
    for s in shape:
        n *= int(s)
    out = torch.empty(n, dtype=dtype, device=device)
    pos = 0
    while pos < n:
        m = min(chunk, n - pos)
        # pairs covering elements [pos, pos+m); pos is kept even
        p0 = pos // 2
        npairs = (m + 1) // 2
        pidx = torch.arange(p0, p0 + npairs, dtype=torch.int64, device=device)
        u1 = uniform01(seed, 2 * pidx)
        u2 = uniform01(seed, 2 * pidx + 1)
        rad = torch.sqrt(-2.0 * torch.log(u1))
        ang = (2.0 * math.pi) * u2
        z = torch.stack((rad * torch.cos(ang), rad * torch.sin(ang)), dim=1).reshape(-1)[:m]
        out[pos:pos + m] = (z * std).to(torch.float32).to(dtype)
        pos += m
        if pos % 2:  # keep chunks pair-aligned (only the last chunk can be odd)
            break
    return out.reshape(*shape)


def permutation(seed: int, n: int) -> torch.Tensor:
    """Seeded permutation of 0..n-1 (argsort of hashed keys), on the CPU."""
    keys = hash_u64(seed, torch.arange(n, dtype=torch.int64))
    # sort by the unsigned value: flip the sign bit so signed order == unsigned order
    return torch.argsort(keys ^ _s64(1 << 63), stable=True)
