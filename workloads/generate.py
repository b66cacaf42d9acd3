"""Seeded synthetic inputs (host side, numpy only).

Every value is a function of (seed, t, k, tensor list) alone, so any consumer
can regenerate exactly the same bits in any order.  Nothing here belongs to the
method: these are the *inputs* the path consumes (initial parameters and
per-step per-worker gradients), standing in for what back-propagation on the
paper's datasets would supply.
"""
from __future__ import annotations

from typing import List, Sequence

import numpy as np

from .shapes import TensorSpec


def _rng(seed: int, stream: int) -> np.random.Generator:
    # numpy's counter-based Philox bit generator, keyed by (seed, stream)
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(stream)]))


def init_params_host(tensors: Sequence[TensorSpec], seed: int, std: float) -> np.ndarray:
    """Flat float32 vector holding the initial model x^(0) (tensors concatenated
    in list order).  "normal": N(0, std^2); "kaiming": N(0, 2/fan_in);
    "ones"/"zeros": constants (normalisation scales / biases).
    """
    P = sum(t.numel for t in tensors)
    out = np.empty(P, dtype=np.float32)
    off = 0
    for j, t in enumerate(tensors):
        n = t.numel
        if t.init == "normal":
            out[off:off + n] = _rng(seed, j).standard_normal(n, dtype=np.float32) * np.float32(std)
        elif t.init == "kaiming":
            s = np.float32(np.sqrt(2.0 / t.fan_in))
            out[off:off + n] = _rng(seed, j).standard_normal(n, dtype=np.float32) * s
        elif t.init == "ones":
            out[off:off + n] = 1.0
        elif t.init == "zeros":
            out[off:off + n] = 0.0
        else:
            raise ValueError(t.init)
        off += n
    return out


def grads_host(P: int, seed: int, t: int, k: int, std: float,
               out: np.ndarray | None = None) -> np.ndarray:
    """Gradient of worker k at step t: P i.i.d. N(0, std^2) float32 values."""
    g = _rng(seed, (int(t) << 16) | int(k)).standard_normal(P, dtype=np.float32)
    g *= np.float32(std)
    if out is not None:
        out[...] = g
        return out
    return g


def bf16_bits_from_f32_host(a: np.ndarray) -> np.ndarray:
    """Make bf16 *inputs* from float32 samples by dropping the low 16 bits.

    Truncation keeps the generator free of any rounding rule the method itself
    uses; the result is an exactly representable bf16 value whose bit pattern
    is returned as uint16.
    """
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def sample_indices(tensors: Sequence[TensorSpec], n_random: int, seed: int,
                   edge: int = 8) -> np.ndarray:
    """Sorted unique flat indices: the first and last `edge` elements of every
    tensor plus `n_random` uniformly drawn positions."""
    P = sum(t.numel for t in tensors)
    idx: List[np.ndarray] = []
    off = 0
    for t in tensors:
        n = t.numel
        e = min(edge, n)
        idx.append(np.arange(off, off + e))
        idx.append(np.arange(off + n - e, off + n))
        off += n
    if n_random > 0:
        idx.append(_rng(seed, 0xFFFF).integers(0, P, size=n_random))
    return np.unique(np.concatenate(idx)).astype(np.int64)
