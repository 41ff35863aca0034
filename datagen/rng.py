"""Counter-based seeded random numbers, bit-identical on CPU and CUDA.

Every sample is a pure function of (stream key, element index): a 32-bit integer
hash picks a quantile of the standard normal from a table that is always built
on the CPU in float64.  Only integer ops and individually rounded fp32 mul/add
are used after that, so a tensor generated on the GPU holds exactly the bits the
CPU generator gives for the same key.  This module draws random inputs only; it
holds none of the method's arithmetic and is the one module that both the CPU
oracle's tests and the CUDA path's tests/bench may import.
"""
from __future__ import annotations

import torch

_M32 = 0xFFFFFFFF
_MULT = 0x45D9F3B  # < 2**27, so a 32-bit value times it stays inside int64
_GOLD = 0x9E3779B9

_TABLE_BITS = 16
_tables: dict[str, tuple[torch.Tensor, torch.Tensor]] = {}


def _mix_int(x: int) -> int:
    x &= _M32
    x = (((x >> 16) ^ x) * _MULT) & _M32
    x = (((x >> 16) ^ x) * _MULT) & _M32
    return ((x >> 16) ^ x) & _M32


def stream_key(seed: int, *words: int) -> tuple[int, int]:
    """Fold (seed, tag words...) into the two 32-bit keys of one random stream."""
    k = _mix_int(seed ^ 0x51ED270B)
    for w in words:
        k = _mix_int((k + _GOLD) & _M32 ^ _mix_int(int(w) & _M32))
    return k, _mix_int(k ^ 0xA5A5A5A5)


def _mix_t(x: torch.Tensor) -> torch.Tensor:
    # x: int64 tensor holding values in [0, 2**32)
    x = (((x >> 16) ^ x) * _MULT) & _M32
    x = (((x >> 16) ^ x) * _MULT) & _M32
    return (x >> 16) ^ x


def uniform_bits(n: int, key: tuple[int, int], device="cpu", offset: int = 0) -> torch.Tensor:
    """n 32-bit hash values (as int64) for element indices offset .. offset+n-1."""
    if offset + n > (1 << 32):
        raise ValueError("one stream addresses at most 2**32 elements")
    idx = torch.arange(offset, offset + n, dtype=torch.int64, device=device)
    a = _mix_t(idx ^ key[0])
    return _mix_t(((a + key[1]) & _M32) ^ (idx >> 7))


def _normal_table(device) -> tuple[torch.Tensor, torch.Tensor]:
    dev = str(torch.device(device))
    if dev not in _tables:
        n = 1 << _TABLE_BITS
        p = torch.arange(n + 1, dtype=torch.float64) / n
        lo = 2.0 ** -(_TABLE_BITS + 1)
        q = torch.special.ndtri(p.clamp(lo, 1.0 - lo))
        base = q[:-1].to(torch.float32)
        step = (q[1:] - q[:-1]).to(torch.float32)
        _tables[dev] = (base.to(device), step.to(device))
    return _tables[dev]


def normal(n: int, key: tuple[int, int], device="cpu", offset: int = 0,
           chunk: int = 1 << 25) -> torch.Tensor:
    """n standard-normal fp32 samples (truncated near +-4.3 sigma)."""
    base, step = _normal_table(device)
    out = torch.empty(n, dtype=torch.float32, device=device)
    for s in range(0, n, chunk):
        m = min(chunk, n - s)
        r = uniform_bits(m, key, device, offset + s)
        i = r >> 16
        frac = (r & 0xFFFF).to(torch.float32) * (1.0 / 65536.0)
        out[s:s + m] = torch.add(base[i], torch.mul(frac, step[i]))
    return out


def uniform_int(n: int, high: int, key: tuple[int, int], device="cpu") -> torch.Tensor:
    """n integers in [0, high) (high <= 2**16; slight modulo bias is irrelevant here)."""
    return (uniform_bits(n, key, device) >> 8) % high


def uniform01(n: int, key: tuple[int, int], device="cpu") -> torch.Tensor:
    """n float64 samples in [0, 1) with 32 bits of resolution."""
    return uniform_bits(n, key, device).to(torch.float64) / float(1 << 32)
