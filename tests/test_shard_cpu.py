"""Parameter-axis sharding: the cut of the tensor list, and the property it rests on --
Algorithm 1 run independently on disjoint slices of all K replicas (same seed) gives exactly
the slices of the unsharded run -- checked with the CPU oracle."""
import numpy as np
import pytest

import oracle
from paper_2504_18454_b200.shard import shard_numel, shard_ranges

RAGGED = [1, 3, 7, 1001, 4095, 4096, 4097, 0, 5, 12289, 8]


@pytest.mark.parametrize("world", [1, 2, 3, 8])
@pytest.mark.parametrize("numel", [RAGGED, [1 << 16], [5], [0, 0, 9000]])
def test_pieces_cover_every_element_exactly_once_in_order(numel, world):
    seen = []
    for rank in range(world):
        pieces = shard_ranges(numel, rank, world, align=64)
        assert shard_numel(numel, rank, world, align=64) == [b - a for _, a, b in pieces]
        for j, a, b in pieces:
            assert 0 <= a < b <= numel[j]
            seen += [(j, i) for i in range(a, b)]
    assert seen == [(j, i) for j, n in enumerate(numel) for i in range(n)]


def test_boundaries_are_aligned_and_sizes_balanced():
    numel = [100000, 33, 70001]
    total, world, align = sum(numel), 4, 1024
    sizes = [sum(shard_numel(numel, r, world, align)) for r in range(world)]
    assert sum(sizes) == total and max(sizes) - min(sizes[:-1]) <= align and all(s % align == 0 for s in sizes[:-1])
    with pytest.raises(ValueError):
        shard_ranges(numel, 4, 4)


@pytest.mark.parametrize("inner,precision", [(0, 0), (1, 1)])
def test_slices_run_independently_equal_the_slices_of_the_whole_run(inner, precision):
    K, world, H, T = 4, 3, 3, 7
    numel = [5000, 17, 3000]
    P = sum(numel)
    rng = np.random.default_rng(3)
    x0 = (rng.standard_normal((K, P)) * 0.02).astype(np.float32)
    kw = dict(K=K, H=H, p=0.3, inner=inner, momentum=0.9 if inner else 0.0, seed=11, precision=precision)
    whole = oracle.Oracle(x0, dtype="f32", **kw)
    starts = np.concatenate([[0], np.cumsum(numel)])
    idx = [np.concatenate([np.arange(starts[j] + a, starts[j] + b) for j, a, b in shard_ranges(numel, r, world, 64)])
           for r in range(world)]
    parts = [oracle.Oracle(x0[:, ix], dtype="f32", **kw) for ix in idx]
    for t in range(T):
        g = (rng.standard_normal((K, P)) * 0.01).astype(np.float32)
        if precision:
            g = (g.view(np.uint32) >> 16).astype(np.uint16)
        whole.step(g, 1e-3, 16.0)
        for part, ix in zip(parts, idx):
            part.step(np.ascontiguousarray(g[:, ix]), 1e-3, 16.0)
    for part, ix in zip(parts, idx):
        assert np.array_equal(part.x, whole.x[:, ix]) and np.array_equal(part.m, whole.m[:, ix])
        assert np.array_equal(part.xg, whole.xg[ix]) and np.array_equal(part.u, whole.u[ix])
        assert list(part.s) == list(whole.s) and part.n_outer == whole.n_outer == 2
