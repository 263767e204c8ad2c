"""Counter-based seeded generator for synthetic tensors.

Element ``j`` of stream ``t`` under seed ``s`` is a pure function of ``(s, t, j)``:
a SplitMix64-style finaliser applied twice (first to the key, then to key + counter).
All arithmetic is wrapping int64, so the same bits come out on the CPU and on a GPU.

Normals are drawn by inverse CDF from the top 16 bits of the hash through a 65536-entry
table (built once, in float64, on the host), so no transcendental function is evaluated
per element and the values do not depend on the device that generates them.

This module holds no arithmetic of the decoding method: it only makes inputs, which are
handed bit-for-bit to whichever implementation consumes them.
"""
from __future__ import annotations

import functools

import numpy as np
import torch

_GOLDEN = -7046029254386353131   # 0x9E3779B97F4A7C15 as int64
_MUL1 = -4658895280553007687     # 0xBF58476D1CE4E5B9 as int64
_MUL2 = -7723592293110705685     # 0x94D049BB133111EB as int64


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of an int64 tensor (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix(z: torch.Tensor) -> torch.Tensor:
    z = z + _GOLDEN
    z = (z ^ _lsr(z, 30)) * _MUL1
    z = (z ^ _lsr(z, 27)) * _MUL2
    return z ^ _lsr(z, 31)


def _key(seed: int, stream: int, device) -> torch.Tensor:
    k = torch.tensor([(int(seed) << 32) + int(stream)], dtype=torch.int64, device=device)
    return _mix(k)


def hash_u64(seed: int, stream: int, n: int, device="cpu", start: int = 0) -> torch.Tensor:
    """n hashed 64-bit words (as int64) for counters start..start+n-1."""
    idx = torch.arange(start, start + n, dtype=torch.int64, device=device)
    return _mix(_key(seed, stream, device) + idx * _GOLDEN)


@functools.lru_cache(maxsize=None)
def _normal_table_np() -> np.ndarray:
    from scipy.special import ndtri
    u = (np.arange(65536, dtype=np.float64) + 0.5) / 65536.0
    return ndtri(u)


_TABLES: dict = {}


def _normal_table(device) -> torch.Tensor:
    key = str(device)
    if key not in _TABLES:
        _TABLES[key] = torch.from_numpy(_normal_table_np()).to(device)
    return _TABLES[key]


def normal(seed: int, stream: int, shape, scale: float = 1.0, device="cpu",
           dtype=torch.float64, chunk: int = 1 << 24) -> torch.Tensor:
    """N(0, scale^2) tensor of the given shape (65536-level inverse-CDF normals)."""
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=dtype, device=device)
    table = _normal_table(device)
    for s in range(0, n, chunk):
        m = min(chunk, n - s)
        h = hash_u64(seed, stream, m, device, start=s)
        out[s:s + m] = (table[_lsr(h, 48)] * scale).to(dtype)
    return out.reshape(shape)


def normal_bf16(seed: int, stream: int, shape, scale: float = 1.0, device="cpu") -> torch.Tensor:
    """N(0, scale^2) rounded once (round-to-nearest-even) to bfloat16."""
    return normal(seed, stream, shape, scale, device, dtype=torch.float32).to(torch.bfloat16)


def integers(seed: int, stream: int, n: int, lo: int, hi: int, device="cpu") -> torch.Tensor:
    """n integers uniform in [lo, hi) (modulo of 62 hashed bits; bias < 2^-40 for small ranges)."""
    h = _lsr(hash_u64(seed, stream, n, device), 2)
    return (h % (hi - lo)) + lo


def uniform(seed: int, stream: int, n: int, device="cpu") -> torch.Tensor:
    """n float64 uniforms in [0, 1) with 53 random bits."""
    h = _lsr(hash_u64(seed, stream, n, device), 11)
    return h.to(torch.float64) * (1.0 / (1 << 53))
