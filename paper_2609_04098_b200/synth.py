"""Seeded synthetic inputs for the NVFP4 W4A4 linear-layer path.

This module only *draws numbers*: a counter-based generator keyed by
(seed, tensor id, element index), a Box-Muller transform and a round to
bf16.  It holds none of the NVFP4 arithmetic (no amax, no scales, no codes),
so the CPU oracle and the CUDA path can both be fed from it without sharing
any of the method.

All tensors are returned as ``numpy.uint16`` arrays holding bf16 bit patterns
(row-major).  ``to_torch_bf16`` reinterprets one as a ``torch.bfloat16`` tensor.

The shapes and statistics follow the paper's model (hidden size 5120, fused
GDN in-projection with 48-wide gate projections, near-Gaussian weights,
activations with a few hot channels far above the median channel) because the
checkpoint and captured activations the paper measured on are not available.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
from typing import List, Sequence, Tuple

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_TWO_PI = 6.283185307179586
_CHUNK = 1 << 22  # elements per work item (even, so Box-Muller pairs never straddle)


def _mix(z: np.ndarray) -> np.ndarray:
    """64-bit finaliser (xor-shift-multiply); wraps modulo 2**64."""
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _key(seed: int, tensor_id: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = _mix(np.array([np.uint64(seed) * _GOLDEN + np.uint64(tensor_id)], dtype=np.uint64))
        k = _mix(k + np.uint64(stream) * _M2)
    return k[0]


def uniform_u64(seed: int, tensor_id: int, stream: int, start: int, count: int) -> np.ndarray:
    """``count`` 64-bit words for counters ``start .. start+count-1``; any
    chunking of the counter range gives the same words."""
    with np.errstate(over="ignore"):
        ctr = np.arange(start, start + count, dtype=np.uint64)
        return _mix(_key(seed, tensor_id, stream) + ctr * _GOLDEN)


def _unit(u: np.ndarray) -> np.ndarray:
    """uint64 -> float64 in (0, 1)."""
    return ((u >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def _normal_chunk(seed: int, tensor_id: int, start: int, count: int) -> np.ndarray:
    """Standard normals for flat element indices start..start+count-1 (start even)."""
    assert start % 2 == 0
    npair = (count + 1) // 2
    u1 = _unit(uniform_u64(seed, tensor_id, 0, start // 2, npair))
    u2 = _unit(uniform_u64(seed, tensor_id, 1, start // 2, npair))
    r = np.sqrt(-2.0 * np.log(u1))
    out = np.empty(2 * npair, dtype=np.float64)
    out[0::2] = r * np.cos(_TWO_PI * u2)
    out[1::2] = r * np.sin(_TWO_PI * u2)
    return out[:count]


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round to bf16 (nearest even) through float32; returns uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _threads() -> int:
    import os
    return max(1, min(32, os.cpu_count() or 1))


def _fill(total: int, fn) -> np.ndarray:
    """Evaluate ``fn(start, count) -> uint16[count]`` over [0, total) in threads."""
    out = np.empty(total, dtype=np.uint16)
    spans = [(s, min(_CHUNK, total - s)) for s in range(0, total, _CHUNK)]

    def work(span):
        s, c = span
        out[s:s + c] = fn(s, c)

    if len(spans) <= 1:
        for sp in spans:
            work(sp)
    else:
        with ThreadPoolExecutor(max_workers=_threads()) as ex:
            list(ex.map(work, spans))
    return out


def hot_columns(seed: int, tensor_id: int, K: int, count: int) -> np.ndarray:
    """A fixed, seed-determined set of ``count`` distinct column indices."""
    if count <= 0:
        return np.zeros(0, dtype=np.int64)
    order = np.argsort(uniform_u64(seed, tensor_id, 2, 0, K), kind="stable")
    return np.sort(order[:count].astype(np.int64))


def activations(seed: int, tensor_id: int, M: int, K: int, *, n_hot: int = 2,
                hot_scale: float = 50.0, spike_p: float = 0.0,
                spike_value: float = 2000.0) -> np.ndarray:
    """bf16 [M, K]: N(0,1) base, ``n_hot`` seed-chosen columns multiplied by
    ``hot_scale``, then each entry independently replaced with probability
    ``spike_p`` by +/-``spike_value`` (sign drawn from the seed)."""
    cols = hot_columns(seed, tensor_id, K, n_hot)
    colscale = np.ones(K, dtype=np.float64)
    colscale[cols] = hot_scale
    thresh = np.uint64(min(int(spike_p * 2.0 ** 64), 2 ** 64 - 1)) if spike_p > 0 else None

    def fn(start, count):
        x = _normal_chunk(seed, tensor_id, start, count)
        k = (np.arange(start, start + count, dtype=np.int64) % K)
        x *= colscale[k]
        if thresh is not None:
            u = uniform_u64(seed, tensor_id, 3, start, count)
            hit = u < thresh
            sign = np.where((u & np.uint64(1)) == 0, 1.0, -1.0)
            x = np.where(hit, sign * spike_value, x)
        return f64_to_bf16_bits(x)

    return _fill(M * K, fn).reshape(M, K)


@dataclass(frozen=True)
class Segment:
    """A fused module's slice of output columns (= rows of the weight matrix)."""
    name: str
    begin: int
    count: int
    std: float = 0.02


def make_segments(spec: Sequence[Tuple[str, int, float]]) -> List[Segment]:
    segs, pos = [], 0
    for name, count, std in spec:
        segs.append(Segment(name, pos, count, std))
        pos += count
    return segs


def weights(seed: int, tensor_id: int, segments: Sequence[Segment], K: int) -> np.ndarray:
    """bf16 [N, K] with N = sum of segment sizes; rows of segment j ~ N(0, std_j)."""
    N = sum(s.count for s in segments)
    rowstd = np.empty(N, dtype=np.float64)
    for s in segments:
        rowstd[s.begin:s.begin + s.count] = s.std

    def fn(start, count):
        x = _normal_chunk(seed, tensor_id, start, count)
        n = np.arange(start, start + count, dtype=np.int64) // K
        return f64_to_bf16_bits(x * rowstd[n])

    return _fill(N * K, fn).reshape(N, K)


# ----------------------------------------------------------------------------
# The benchmark configurations (shapes from the paper's model; see module doc).
# ----------------------------------------------------------------------------
GDN_SEGMENTS = (("q", 2048, 0.02), ("k", 2048, 0.02), ("v", 6144, 0.02),
                ("z", 6144, 0.02), ("a", 48, 0.2), ("b", 48, 0.2))
HIDDEN = 5120
MLP_INNER = 17408


def config1(seed: int = 0):
    """Single linear 128x512 -> 256, two hot channels x50."""
    segs = make_segments((("w", 256, 0.02),))
    return activations(seed, 101, 128, 512, n_hot=2, hot_scale=50.0), weights(seed, 102, segs, 512), segs


def config2_activations(seed: int = 0, M: int = 8192, K: int = HIDDEN) -> np.ndarray:
    """Heavy-tailed activations: 0.5 % hot channels x100, 1e-4 spikes of +/-2000."""
    return activations(seed, 201, M, K, n_hot=int(round(0.005 * K)), hot_scale=100.0,
                       spike_p=1e-4, spike_value=2000.0)


def prefill_activations(seed: int, tensor_id: int, M: int, K: int) -> np.ndarray:
    """Activations "as config 1": N(0,1) with two hot channels x50."""
    return activations(seed, tensor_id, M, K, n_hot=2, hot_scale=50.0)


def to_torch_bf16(bits: np.ndarray):
    """Reinterpret a uint16 bit-pattern array as a torch.bfloat16 CPU tensor (no copy)."""
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
