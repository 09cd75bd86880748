"""Counter-based random numbers for the synthetic workloads.

Every value is a pure function of (seed, stream, index), so any slice of any
array can be produced on its own, on the CPU or on a GPU, without generating
what comes before it.  The integer stream is SplitMix64 (Steele, Lea, Flood,
"Fast splittable pseudorandom number generators", OOPSLA 2014) applied to a
counter; everything is written with torch int64 arithmetic, which wraps
modulo 2**64 on both devices.

This module holds no arithmetic of the parameter-server method itself: it is
the one piece of code that both the CUDA library's callers and the CPU oracle's
callers may share.
"""
from __future__ import annotations

import math

import numpy as np
import torch

_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_MUL1 = 0xBF58476D1CE4E5B9
_MUL2 = 0x94D049BB133111EB


def _s64(x: int) -> int:
    """Python int (mod 2**64) -> the signed value torch.int64 holds."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def _mix_int(x: int) -> int:
    x = (x + _GOLDEN) & _M64
    z = x
    z = ((z ^ (z >> 30)) * _MUL1) & _M64
    z = ((z ^ (z >> 27)) * _MUL2) & _M64
    return z ^ (z >> 31)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of an int64 tensor (torch's >> is arithmetic)."""
    return (x >> s) & _s64((1 << (64 - s)) - 1)


def _mix_tensor(x: torch.Tensor) -> torch.Tensor:
    z = x + _s64(_GOLDEN)
    z = (z ^ _lsr(z, 30)) * _s64(_MUL1)
    z = (z ^ _lsr(z, 27)) * _s64(_MUL2)
    return z ^ _lsr(z, 31)


def stream_key(seed: int, stream: int) -> int:
    """Scalar key of one named stream of one seed."""
    return _mix_int(_mix_int(seed & _M64) ^ ((stream * 0xD1B54A32D192ED03) & _M64))


def bits64(seed: int, stream: int, index: torch.Tensor) -> torch.Tensor:
    """64 random bits per entry of `index` (int64 tensor of counters)."""
    assert index.dtype == torch.int64
    return _mix_tensor(index + _s64(stream_key(seed, stream)))


def counter(start: int, count: int, device) -> torch.Tensor:
    return torch.arange(start, start + count, dtype=torch.int64, device=device)


def uniform01(seed: int, stream: int, index: torch.Tensor) -> torch.Tensor:
    """float64 in [0, 1): the top 53 bits of the 64-bit word."""
    return _lsr(bits64(seed, stream, index), 11).to(torch.float64) * (2.0 ** -53)


def uniform_int(seed: int, stream: int, index: torch.Tensor, n: int) -> torch.Tensor:
    """int64 in [0, n) (floor of n * u; n far below 2**53)."""
    return torch.clamp((uniform01(seed, stream, index) * n).to(torch.int64), max=n - 1)


def normal(seed: int, stream: int, index: torch.Tensor, std: float = 1.0) -> torch.Tensor:
    """float64 N(0, std**2) by Box-Muller from two independent words per index."""
    u1 = uniform01(seed, stream, index * 2)
    u2 = uniform01(seed, stream, index * 2 + 1)
    r = torch.sqrt(-2.0 * torch.log1p(-u1))          # 1 - u1 in (0, 1]
    return r * torch.cos((2.0 * math.pi) * u2) * std


def power_law_cdf(n: int, exponent: float) -> np.ndarray:
    """float64 CDF of p(rank) ~ rank**(-exponent), rank = 1..n (entry r-1 = P[rank <= r])."""
    w = np.arange(1, n + 1, dtype=np.float64) ** (-exponent)
    c = np.cumsum(w)
    c /= c[-1]
    c[-1] = 1.0
    return c


def sample_cdf(cdf: torch.Tensor, u: torch.Tensor) -> torch.Tensor:
    """Inverse-CDF sample: smallest r with cdf[r] > u, as int64 in [0, len(cdf))."""
    idx = torch.searchsorted(cdf, u, right=True)
    return torch.clamp(idx, max=cdf.numel() - 1)
