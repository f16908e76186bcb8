"""Seeded synthetic KV payloads: a pure integer function of (seed, stream, element index).

This module only PRODUCES inputs.  It holds none of the operators' arithmetic and is
the one piece of code the CPU oracle's tests and the CUDA path's tests both use, so
that both sides see identical bytes.  Element values are bf16 bit patterns whose
marginal distribution is N(0,1) rounded to bf16 (the KV pools of the workloads are
"seeded N(0,1) rounded to bf16"); the operators treat them as opaque 16-bit payload.

    value16(seed, stream, i) = Q[ top16( mix64( key(seed, stream) + i * ODD ) ) ]

  * mix64 is the splitmix64 output finaliser (two multiply / xor-shift rounds).
  * Q is the 65,536-entry table of N(0,1) quantiles Phi^-1((j + 1/2) / 65536),
    evaluated once in float64 on the CPU, rounded to float32 and then to bf16
    (round to nearest even); no transcendental is ever evaluated on the GPU.
  * stream 0 is a pool's initial image (index = linear index in [L, NB, 2, BS, H, D]);
    stream s >= 1 is the payload of one import/append (index = linear index in its
    [L, 2, n, H, D] transfer buffer).

Because any element can be evaluated on its own, expected values of sampled outputs
at full size never need a second copy of the data.
"""
from __future__ import annotations

import numpy as np

_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_ODD = 0x9E3779B97F4A7C15
_KS = 0xD6E8FEB86659FD93
_KT = 0xA0761D6478BD642F
_MASK = (1 << 64) - 1

_Q = None


def quantile_table() -> np.ndarray:
    """uint16[65536]: bf16 bit patterns of the N(0,1) quantiles (see module docstring)."""
    global _Q
    if _Q is None:
        from scipy.special import ndtri

        q64 = ndtri((np.arange(65536, dtype=np.float64) + 0.5) / 65536.0)
        bits = q64.astype(np.float32).view(np.uint32).astype(np.uint64)
        # float32 -> bf16, round to nearest even on the dropped 16 bits
        rounded = (bits + 0x7FFF + ((bits >> 16) & 1)) >> 16
        _Q = rounded.astype(np.uint16)
    return _Q


def stream_key(seed: int, stream: int) -> int:
    return (seed * _KS + stream * _KT + 0x1234567) & _MASK


def fill_np_at(seed: int, stream: int, idx) -> np.ndarray:
    """uint16 array, same shape as ``idx``: the stream's elements at arbitrary indices."""
    with np.errstate(over="ignore"):
        i = np.asarray(idx).astype(np.uint64)
        x = np.uint64(stream_key(seed, stream)) + i * np.uint64(_ODD)
        x ^= x >> np.uint64(30)
        x *= np.uint64(_M1)
        x ^= x >> np.uint64(27)
        x *= np.uint64(_M2)
        x ^= x >> np.uint64(31)
    return quantile_table()[(x >> np.uint64(48)).astype(np.int64)]


def fill_np(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    """uint16[count]: elements start .. start+count-1 of the given stream (numpy)."""
    return fill_np_at(seed, stream, np.arange(start, start + count, dtype=np.uint64))


def _s64(v: int) -> int:
    """two's-complement int64 value of a uint64 constant"""
    v &= _MASK
    return v - (1 << 64) if v >= (1 << 63) else v


def _lsr(x, s):
    """logical right shift of an int64 tensor (arithmetic shift, then mask)"""
    return (x >> s) & ((1 << (64 - s)) - 1)


def quantile_table_torch(device):
    import torch

    return torch.from_numpy(quantile_table().view(np.int16).copy()).to(device)


def fill_torch_at(key, idx, q):
    """int16 tensor shaped like ``idx``: elements ``idx`` (int64 tensor) of the stream(s) whose key(s) ``key`` is
    an int (one stream) or an int64 tensor broadcastable against ``idx`` (``key_s64`` of each element's stream).
    Wrapping int64 arithmetic; ``q`` = quantile_table_torch(device)."""
    x = idx * _s64(_ODD) + key
    x = x ^ _lsr(x, 30)
    x = x * _s64(_M1)
    x = x ^ _lsr(x, 27)
    x = x * _s64(_M2)
    x = x ^ _lsr(x, 31)
    return q[_lsr(x, 48)]


def key_s64(seed: int, stream: int) -> int:
    """the stream key as a two's-complement int64 (what fill_torch_at adds)"""
    return _s64(stream_key(seed, stream))


def fill_torch(seed: int, stream: int, start: int, count: int, device, out=None, chunk: int = 1 << 26):
    """int16 tensor [count] on ``device`` holding the same bit patterns as fill_np.

    Written with wrapping int64 arithmetic (logical right shifts are an arithmetic
    shift followed by a mask), in chunks so that temporaries stay small.
    """
    import torch

    if out is None:
        out = torch.empty(count, dtype=torch.int16, device=device)
    assert out.numel() == count and out.dtype == torch.int16
    q = quantile_table_torch(device)
    key = key_s64(seed, stream)
    done = 0
    while done < count:
        c = min(chunk, count - done)
        i = torch.arange(start + done, start + done + c, dtype=torch.int64, device=device)
        out[done : done + c] = fill_torch_at(key, i, q)
        done += c
    return out
