"""Seeded synthetic weights and gradients, bit-identical on CPU and GPU.

Every value is a pure function of (seed, stream, element index), so any subset
of elements can be produced on its own, on any device, with the same bits:
a full 61 M-element gradient on the GPU and a few thousand sampled elements of
the same gradient on the CPU agree exactly.  That is achieved by doing all the
randomness in 64-bit integer arithmetic and ending with a single fp32 multiply:

  1. a stream key is derived from (seed, stream kind, learner, push index);
  2. each element index is hashed three times with the SplitMix64 finaliser
     (Steele, Lea, Flood: "Fast splittable pseudorandom number generators",
     OOPSLA 2014);
  3. the twelve 16-bit fields of the three hashes are summed: an Irwin-Hall
     sum, whose distribution is close to normal (excess kurtosis -0.1,
     support +-6 standard deviations);
  4. the centred integer (|x| < 2^24, exact in fp32) is multiplied by
     std / stddev(x) rounded once to fp32.

This stands in for the N(0, std^2) draws of the workloads.  The module holds
no update arithmetic and knows nothing of timestamps or staleness.
"""
from __future__ import annotations

import math
from typing import Optional

import torch

from .layouts import Layout

_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_MUL1 = 0xBF58476D1CE4E5B9
_MUL2 = 0x94D049BB133111EB

STREAM_WEIGHTS = 1
STREAM_GRADIENT = 2

_FIELDS = 12
# x = 2*sum(fields) - FIELDS*65535 has variance FIELDS/3 * (65536^2 - 1)
_X_STD = math.sqrt(_FIELDS / 3.0 * (65536.0 ** 2 - 1.0))
_CHUNK = 1 << 24


def _s64(x: int) -> int:
    """Python int in [0, 2^64) -> the int64 with the same bit pattern."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def mix64_int(z: int) -> int:
    """SplitMix64 finaliser on a Python int (mod 2^64)."""
    z &= _M64
    z = ((z ^ (z >> 30)) * _MUL1) & _M64
    z = ((z ^ (z >> 27)) * _MUL2) & _M64
    return z ^ (z >> 31)


def _lsr(z: torch.Tensor, k: int) -> torch.Tensor:
    """Logical right shift of int64 bit patterns."""
    return (z >> k) & ((1 << (64 - k)) - 1)


def mix64(z: torch.Tensor) -> torch.Tensor:
    """SplitMix64 finaliser on int64 tensors (two's-complement wrap-around)."""
    z = (z ^ _lsr(z, 30)) * _s64(_MUL1)
    z = (z ^ _lsr(z, 27)) * _s64(_MUL2)
    return z ^ _lsr(z, 31)


def stream_key(seed: int, kind: int, a: int = 0, b: int = 0) -> int:
    """64-bit key of one stream: kind (weights / gradient), learner a, push b."""
    k = mix64_int(seed)
    k = mix64_int(k ^ (kind * _GOLDEN & _M64))
    k = mix64_int(k ^ ((a + 1) * _MUL1 & _M64))
    k = mix64_int(k ^ ((b + 1) * _MUL2 & _M64))
    return k


def _field_sum(h: torch.Tensor) -> torch.Tensor:
    """Sum of the four 16-bit fields of each 64-bit pattern."""
    m = 0x0000FFFF0000FFFF
    t = (h & m) + (_lsr(h, 16) & m)          # two 17-bit sums at bits 0 and 32
    return (t & 0xFFFFFFFF) + _lsr(t, 32)


def centred_integers(key: int, index: torch.Tensor) -> torch.Tensor:
    """int64 x(index) with mean 0 and standard deviation _X_STD, |x| < 2^24."""
    base = index * _s64(_GOLDEN) + _s64(key)
    h = mix64(base)
    total = _field_sum(h)
    for r in (1, 2):
        h = mix64(base ^ _s64(mix64_int(key + r)))
        total = total + _field_sum(h)
    return 2 * total - _FIELDS * 65535


def scale_for(std: float) -> float:
    """The fp32 multiplier that gives the centred integers standard deviation std."""
    return float(torch.tensor(std / _X_STD, dtype=torch.float64).to(torch.float32))


def normal_like_at(key: int, index: torch.Tensor, std: float) -> torch.Tensor:
    """fp32 values at the given int64 element indices (any device)."""
    x = centred_integers(key, index).to(torch.float32)
    return x * scale_for(std)


def normal_like(key: int, start: int, count: int, std: float,
                device="cpu", out: Optional[torch.Tensor] = None,
                dtype: torch.dtype = torch.float32) -> torch.Tensor:
    """Elements [start, start+count) of a stream, generated in bounded chunks."""
    if out is None:
        out = torch.empty(count, dtype=dtype, device=device)
    assert out.numel() == count
    for c0 in range(0, count, _CHUNK):
        c1 = min(count, c0 + _CHUNK)
        idx = torch.arange(start + c0, start + c1, dtype=torch.int64, device=out.device)
        out[c0:c1] = normal_like_at(key, idx, std).to(out.dtype)
    return out


def gradient(seed: int, learner: int, push_index: int, num_params: int, std: float,
             dtype: torch.dtype = torch.float32, device="cpu",
             out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """The gradient vector of push number `push_index` of `learner`.

    dtype torch.bfloat16 rounds the fp32 value to nearest-even; both the
    reference and the GPU path then consume those bf16 values.
    """
    key = stream_key(seed, STREAM_GRADIENT, learner, push_index)
    return normal_like(key, 0, num_params, std, device=device, out=out, dtype=dtype)


def gradient_at(seed: int, learner: int, push_index: int, index: torch.Tensor, std: float,
                dtype: torch.dtype = torch.float32) -> torch.Tensor:
    """Selected elements of the same gradient vector."""
    key = stream_key(seed, STREAM_GRADIENT, learner, push_index)
    return normal_like_at(key, index, std).to(dtype)


def _bias_mask(layout: Layout, index: torch.Tensor) -> torch.Tensor:
    mask = torch.zeros_like(index, dtype=torch.bool)
    for seg in layout.segments:
        if seg.is_bias:
            mask |= (index >= seg.offset) & (index < seg.offset + seg.count)
    return mask


def initial_weights(layout: Layout, seed: int, std: float = 0.01, device="cpu") -> torch.Tensor:
    """fp32 initial weights: N(0, std^2)-like for weight segments, 0 for biases."""
    key = stream_key(seed, STREAM_WEIGHTS)
    w = normal_like(key, 0, layout.num_params, std, device=device)
    for seg in layout.segments:
        if seg.is_bias:
            w[seg.offset:seg.offset + seg.count] = 0.0
    return w


def initial_weights_at(layout: Layout, seed: int, index: torch.Tensor, std: float = 0.01) -> torch.Tensor:
    key = stream_key(seed, STREAM_WEIGHTS)
    w = normal_like_at(key, index, std)
    w[_bias_mask(layout, index)] = 0.0
    return w
