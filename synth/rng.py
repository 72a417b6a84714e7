"""Counter-based, integer-only pseudo-random tensors.

Every element is a pure function of (seed, stream, element index), so a tensor
can be produced in any chunking, on the CPU or on a CUDA device, and come out
bit-identical.  The element hash is the published SplitMix64 finaliser
(Steele, Lea & Flood, "Fast splittable pseudorandom number generators", 2014)
applied to ``base + index``.  A pseudo-normal value is the centred sum of the
four 16-bit fields of the hash (Irwin-Hall with four terms), scaled by one fp32
multiplication - there is no transcendental function anywhere, hence nothing
that could round differently on different hardware.
"""
from __future__ import annotations

import math

import torch

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB


def _signed(v: int) -> int:
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def _splitmix64_int(x: int) -> int:
    x = (x + _GOLDEN) & _MASK64
    z = x
    z = ((z ^ (z >> 30)) * _C1) & _MASK64
    z = ((z ^ (z >> 27)) * _C2) & _MASK64
    return z ^ (z >> 31)


def stream_base(seed: int, stream: int) -> int:
    """Scalar base counter of the (seed, stream) pair."""
    return _splitmix64_int(_splitmix64_int(seed & _MASK64) ^ ((stream * 0xD1342543DE82EF95) & _MASK64))


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    # logical shift right on int64 storage
    return (z >> s) & ((1 << (64 - s)) - 1)


def _hash(idx: torch.Tensor, base: int) -> torch.Tensor:
    z = idx + _signed(base + _GOLDEN)
    z = (z ^ _lsr(z, 30)) * _signed(_C1)
    z = (z ^ _lsr(z, 27)) * _signed(_C2)
    return z ^ _lsr(z, 31)


# standard deviation of the centred sum of four independent uniforms on {0..65535}
_IH4_SD = math.sqrt(4.0 * (65536.0 ** 2 - 1.0) / 12.0)
_CHUNK = 1 << 24


def pseudo_normal(seed: int, stream: int, shape, std: float, *, mean: float = 0.0,
                  dtype=torch.float32, device="cpu", offset: int = 0) -> torch.Tensor:
    """Tensor of ``shape`` with element i = mean + std * z(seed, stream, offset + i)."""
    numel = 1
    for s in shape:
        numel *= int(s)
    out = torch.empty(numel, dtype=dtype, device=device)
    base = stream_base(seed, stream)
    scale = float(torch.tensor(std / _IH4_SD, dtype=torch.float32))
    for lo in range(0, numel, _CHUNK):
        hi = min(numel, lo + _CHUNK)
        idx = torch.arange(offset + lo, offset + hi, dtype=torch.int64, device=device)
        h = _hash(idx, base)
        s = (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + _lsr(h, 48)
        v = (s - 131070).to(torch.float32) * scale
        if mean != 0.0:
            v = v + mean
        out[lo:hi] = v.to(dtype)
    return out.view(*shape)


def uniform_ints(seed: int, stream: int, count: int, high: int, *, offset: int = 0) -> torch.Tensor:
    """``count`` int64 values in [0, high) on the CPU."""
    idx = torch.arange(offset, offset + count, dtype=torch.int64)
    h = _hash(idx, stream_base(seed, stream))
    return _lsr(h, 11) % int(high)


def uniform_unit(seed: int, stream: int, count: int, *, offset: int = 0) -> torch.Tensor:
    """``count`` float64 values in [0, 1) on the CPU (53 random bits each)."""
    idx = torch.arange(offset, offset + count, dtype=torch.int64)
    h = _hash(idx, stream_base(seed, stream))
    return _lsr(h, 11).to(torch.float64) / float(1 << 53)
