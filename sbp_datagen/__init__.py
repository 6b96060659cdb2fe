"""Seeded synthetic inputs for the SBP boxing / sharded-operator tests and benchmarks.

This module only *draws numbers*.  It holds none of the arithmetic of the SBP method
(no splitting, reduction, matmul, softmax or gather) and is the single piece of code
that both the CPU oracle's tests and the CUDA path's tests/benchmarks call.

Every value is a pure function of (seed, tensor_id, linear index): a counter is
hashed with the splitmix64 finaliser (Steele, Lea & Flood 2014; Vigna's public
domain constants), mapped to the open interval (0, 1) and then to the requested
distribution.  The functions run on whichever torch device is asked for; a tensor
generated on one device is copied, never regenerated, when the other side needs it
(the transcendental functions used by Box-Muller are not bit-identical across devices).
"""
from __future__ import annotations

import math

import torch

_MASK64 = (1 << 64) - 1


def _s64(v: int) -> int:
    """Two's-complement view of an unsigned 64-bit constant as a Python int."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


_GAMMA = _s64(0x9E3779B97F4A7C15)
_M1 = _s64(0xBF58476D1CE4E5B9)
_M2 = _s64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of int64 lanes (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix(x: torch.Tensor) -> torch.Tensor:
    z = x + _GAMMA
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def _mix_int(x: int) -> int:
    z = (x + 0x9E3779B97F4A7C15) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


def _key(seed: int, tensor_id: int, stream: int) -> int:
    return _s64(_mix_int(_mix_int((seed << 32) ^ tensor_id) + stream))


def _unit(seed: int, tensor_id: int, stream: int, start: int, count: int, device) -> torch.Tensor:
    """count float64 values in the OPEN interval (0,1) for counters start..start+count-1."""
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    h = _mix(idx + _key(seed, tensor_id, stream))
    # 52 random bits + 0.5 is exact in float64, never 0 and never 1.
    return (_lsr(h, 12).to(torch.float64) + 0.5) * (2.0 ** -52)


_CHUNK = 1 << 24


def _fill(shape, dtype, device, fn) -> torch.Tensor:
    n = 1
    for s in shape:
        n *= int(s)
    out = torch.empty(n, dtype=dtype, device=device)
    for start in range(0, n, _CHUNK):
        cnt = min(_CHUNK, n - start)
        out[start:start + cnt] = fn(start, cnt).to(dtype)
    return out.reshape(tuple(int(s) for s in shape))


def uniform(seed: int, tensor_id: int, shape, lo: float, hi: float,
            dtype=torch.float32, device="cpu") -> torch.Tensor:
    """uniform(lo, hi) on the open interval, rounded (RNE) to dtype.  Never emits -0.0."""
    def fn(start, cnt):
        u = _unit(seed, tensor_id, 0, start, cnt, device)
        return lo + (hi - lo) * u
    return _fill(shape, dtype, device, fn)


def normal(seed: int, tensor_id: int, shape, mean: float, std: float,
           dtype=torch.float32, device="cpu") -> torch.Tensor:
    """normal(mean, std) by Box-Muller on two counter streams, rounded (RNE) to dtype."""
    def fn(start, cnt):
        u1 = _unit(seed, tensor_id, 1, start, cnt, device)
        u2 = _unit(seed, tensor_id, 2, start, cnt, device)
        z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
        return mean + std * z
    return _fill(shape, dtype, device, fn)


def integers(seed: int, tensor_id: int, shape, lo: int, hi: int, device="cpu") -> torch.Tensor:
    """int64 values uniform over [lo, hi)."""
    def fn(start, cnt):
        u = _unit(seed, tensor_id, 3, start, cnt, device)
        return (torch.floor(u * float(hi - lo)).to(torch.int64) + lo).clamp_(lo, hi - 1)
    return _fill(shape, torch.int64, device, fn)


def small_integers(seed: int, tensor_id: int, shape, lo: int, hi: int,
                   dtype=torch.float32, device="cpu") -> torch.Tensor:
    """Integer-valued floating tensor in [lo, hi): sums/products of these stay exact."""
    return integers(seed, tensor_id, shape, lo, hi, device).to(dtype)


_ZIPF_CACHE: dict = {}


def zipf_ids(seed: int, tensor_id: int, shape, n_rows: int, s: float = 1.05,
             device="cpu") -> torch.Tensor:
    """int64 row ids with Zipf(s) popularity over n_rows ranks.

    rank (0-based) is drawn by inverse CDF from an fp64 cumulative table; the rank is
    then spread over the table by row = rank * 0x9E3779B1 mod n_rows (a bijection when
    n_rows is a power of two, since the multiplier is odd), the way hashed categorical
    ids land in CTR pipelines, so hot rows are not all in the first shard.
    """
    key = (n_rows, float(s), str(device))
    cdf = _ZIPF_CACHE.get(key)
    if cdf is None:
        w = torch.arange(1, n_rows + 1, dtype=torch.float64, device=device).pow_(-s)
        cdf = torch.cumsum(w, 0)
        cdf /= cdf[-1].clone()
        _ZIPF_CACHE.clear()
        _ZIPF_CACHE[key] = cdf
    power_of_two = (n_rows & (n_rows - 1)) == 0

    def fn(start, cnt):
        u = _unit(seed, tensor_id, 4, start, cnt, device)
        rank = torch.searchsorted(cdf, u).clamp_(0, n_rows - 1)
        if power_of_two:
            return (rank * 0x9E3779B1) & (n_rows - 1)
        return rank
    return _fill(shape, torch.int64, device, fn)
