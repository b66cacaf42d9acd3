"""Parameter-axis sharding of a tensor list over several GPUs.

Every operation of the path -- inner optimizer step, pull, K-way average, outer update,
broadcast -- is elementwise in the parameter index, and the branch decisions are a pure
function of (seed, t, k).  A GPU that holds elements [a, b) of ALL K replica slots (and of
x and u) can therefore run Algorithm 1 on its slice with no exchange at all: G GPUs, each
with its own context over P/G elements and the same seed, compute exactly the slices of
the single-GPU result.  (Global-norm gradient clipping is the exception: its norm runs over
the whole gradient and would need one all-reduce of K sums of squares per step.)

This module only cuts the tensor list; it holds no arithmetic.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

Piece = Tuple[int, int, int]          # (tensor index, first element, one past the last element)


def shard_ranges(numel: Sequence[int], rank: int, world: int, align: int = 1024) -> List[Piece]:
    """The pieces of the tensor list that `rank` of `world` owns.

    The concatenated list of sum(numel) elements is cut into `world` contiguous ranges of
    nearly equal size whose boundaries are multiples of `align` elements of the concatenated
    index (with tensors packed back to back in 16-byte-aligned buffers every slice then stays
    16-byte aligned for every element type; slices of separately allocated tensors may lose the
    alignment and take the library's scalar path, with identical results; the last range takes
    the remainder).  Returns, in order, (tensor, start, stop) for every tensor the range touches.
    """
    if world < 1 or not 0 <= rank < world or align < 1:
        raise ValueError("need 0 <= rank < world and align >= 1")
    total = int(sum(numel))
    per = -(-total // world)                       # ceil
    per = -(-per // align) * align                 # round up to the alignment
    lo, hi = min(total, rank * per), min(total, (rank + 1) * per)
    pieces: List[Piece] = []
    off = 0
    for j, n in enumerate(numel):
        a, b = max(lo, off), min(hi, off + int(n))
        if a < b:
            pieces.append((j, a - off, b - off))
        off += int(n)
    return pieces


def shard_span(numel: Sequence[int], rank: int, world: int, align: int = 1024) -> Tuple[int, int]:
    """[lo, hi) of the concatenated element index that `rank` owns (the range `shard_ranges` cuts up)."""
    if world < 1 or not 0 <= rank < world or align < 1:
        raise ValueError("need 0 <= rank < world and align >= 1")
    total = int(sum(numel))
    per = -(-total // world)
    per = -(-per // align) * align
    return min(total, rank * per), min(total, (rank + 1) * per)


def shard_numel(numel: Sequence[int], rank: int, world: int, align: int = 1024) -> List[int]:
    """Element counts of the pieces of `shard_ranges` (the tensor list a rank's context is built on)."""
    return [b - a for _, a, b in shard_ranges(numel, rank, world, align)]
