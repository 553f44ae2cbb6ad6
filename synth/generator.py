"""Counter-based generator of bf16 N(0,1) inputs and of head scores / masks.

Every value is a pure function of integers:

    bits(seed, stream, layer, t, b, head, d) = TABLE[ top16( H(...) ) ]

where ``H`` chains the splitmix64 finaliser (Steele, Lea & Flood 2014) over the
coordinates and ``TABLE[i]`` is the bf16 rounding of the standard-normal quantile at
``(i + 0.5) / 65536``.  After the table is built everything is 64-bit integer
arithmetic carried out by torch on whichever device is asked for, so the CPU and the
CUDA fills are bit-identical and one (layer, b, head) history can be regenerated
alone.

The head mask recipe: scores ``u ~ U[0,1)`` over all ``layers * kv_heads`` heads from
the same hash; the ``round_half_up(frac * layers * kv_heads)`` lowest-scoring heads
are compressed (the highest-scoring heads keep their full cache); ties keep the lower
flat index full.
"""
from __future__ import annotations

import functools

import numpy as np
import torch

STREAM_K = 0
STREAM_V = 1
STREAM_Q = 2
_STREAM_SCORE = 3


def _s64(x: int) -> int:
    """Two's-complement view of an unsigned 64-bit constant as a Python int64 value."""
    x &= (1 << 64) - 1
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_M1 = _s64(0xBF58476D1CE4E5B9)
_M2 = _s64(0x94D049BB133111EB)
_ODD_T = _s64(0xD6E8FEB86659FD93)
_ODD_E = _s64(0xA0761D6478BD642F)
_ODD_S = _s64(0xE7037ED1A0B428DB)


def _lsr(x: torch.Tensor, k: int) -> torch.Tensor:
    """Logical shift right of int64 lanes (torch's >> is arithmetic)."""
    return (x >> k) & ((1 << (64 - k)) - 1)


def _mix64(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 output function on int64 lanes (wrap-around arithmetic)."""
    x = x + _GOLDEN
    x = (x ^ _lsr(x, 30)) * _M1
    x = (x ^ _lsr(x, 27)) * _M2
    return x ^ _lsr(x, 31)


def _scalar(v: int, device) -> torch.Tensor:
    return torch.tensor([_s64(v)], dtype=torch.int64, device=device)


def _stream_key(seed: int, stream: int, layer: int, device) -> torch.Tensor:
    k = _mix64(_scalar(seed, device) * _ODD_S + stream)
    return _mix64(k + layer)


@functools.lru_cache(maxsize=None)
def _normal_table_cpu() -> torch.Tensor:
    p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
    z = torch.special.ndtri(p)
    return z.to(torch.bfloat16).view(torch.int16).clone()


_TABLE_CACHE: dict = {}


def normal_table(device="cpu") -> torch.Tensor:
    """int16[65536]: bf16 bit patterns of the N(0,1) quantiles at (i+0.5)/65536.

    Always built on the CPU in float64 and then moved, so every device sees the same
    table."""
    dev = torch.device(device)
    key = str(dev)
    if key not in _TABLE_CACHE:
        _TABLE_CACHE[key] = _normal_table_cpu().to(dev)
    return _TABLE_CACHE[key]


def _bits_from_keys(tkey: torch.Tensor, elem: torch.Tensor, device) -> torch.Tensor:
    h = _mix64(tkey.reshape(-1, 1) + elem.reshape(1, -1) * _ODD_E)
    idx = _lsr(h, 48)
    return normal_table(device)[idx]


def rows(seed: int, stream: int, layer: int, t0: int, t1: int,
         batch: int, heads: int, head_dim: int, device="cpu") -> torch.Tensor:
    """bf16 tensor [t1-t0, batch, heads, head_dim] for tokens t0..t1-1 of one layer."""
    dev = torch.device(device)
    lkey = _stream_key(seed, stream, layer, dev)
    t = torch.arange(t0, t1, dtype=torch.int64, device=dev)
    tkey = _mix64(lkey + t * _ODD_T)
    elem = torch.arange(batch * heads * head_dim, dtype=torch.int64, device=dev)
    bits = _bits_from_keys(tkey, elem, dev)
    return bits.view(torch.bfloat16).reshape(t1 - t0, batch, heads, head_dim)


def unit_rows(seed: int, stream: int, layer: int, t0: int, t1: int,
              batch: int, heads: int, head_dim: int, b: int, head: int,
              device="cpu") -> torch.Tensor:
    """bf16 tensor [t1-t0, head_dim]: the slice ``rows(...)[:, b, head, :]`` computed alone."""
    dev = torch.device(device)
    lkey = _stream_key(seed, stream, layer, dev)
    t = torch.arange(t0, t1, dtype=torch.int64, device=dev)
    tkey = _mix64(lkey + t * _ODD_T)
    base = (b * heads + head) * head_dim
    elem = torch.arange(base, base + head_dim, dtype=torch.int64, device=dev)
    bits = _bits_from_keys(tkey, elem, dev)
    return bits.view(torch.bfloat16).reshape(t1 - t0, head_dim)


def bf16_bits_to_float(bits: np.ndarray) -> np.ndarray:
    """uint16/int16 bf16 bit patterns -> float32 values (exact)."""
    u = np.asarray(bits).astype(np.uint16).astype(np.uint32) << 16
    return u.view(np.float32)


def head_scores(seed: int, layers: int, kv_heads: int) -> np.ndarray:
    """float64[layers*kv_heads] in [0,1): 53-bit uniform scores standing in for learned gates."""
    key = _mix64(_scalar(seed, "cpu") * _ODD_S + _STREAM_SCORE)
    idx = torch.arange(layers * kv_heads, dtype=torch.int64)
    h = _mix64(key + idx * _ODD_T)
    return (_lsr(h, 11).to(torch.float64) / float(1 << 53)).numpy()


def head_mask(seed: int, layers: int, kv_heads: int, frac_compressed: float) -> np.ndarray:
    """uint8[layers*kv_heads]: 1 = full cache, 0 = compressed (global selection over layers)."""
    total = layers * kv_heads
    n_comp = int(np.floor(frac_compressed * total + 0.5))
    n_comp = max(0, min(total, n_comp))
    u = head_scores(seed, layers, kv_heads)
    # ascending score; among equal scores the HIGHER flat index is compressed first
    order = sorted(range(total), key=lambda i: (u[i], -i))
    mask = np.ones(total, dtype=np.uint8)
    for i in order[:n_comp]:
        mask[i] = 0
    return mask
