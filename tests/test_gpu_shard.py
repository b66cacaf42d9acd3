"""Parameter-axis sharding on the GPU: contexts built over the slices that each rank of a
G-GPU job would own (run here one after the other on one GPU; they never wait on each other)
reproduce the slices of the single-context run bit for bit, with no exchange between them."""
import numpy as np
import pytest

import workloads as W
from workloads.configs import WorkloadConfig
from paper_2504_18454_b200.shard import shard_ranges
from _harness import GpuRun

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("inner,precision", [(0, 0), (0, 1), (1, 0)])
def test_sharded_contexts_equal_the_slices_of_the_whole_context(inner, precision):
    numel = [4096 * 5 + 8, 4096 * 2, 1000, 24]
    P, K, world = sum(numel), 4, 3
    cfg = WorkloadConfig(name="shard", shape=lambda: [], K=K, H=3, p=0.3, eta=16.0, lr=1e-3, T=7, inner=inner,
                         precision=precision, momentum=0.9 if inner else 0.0)
    rng = np.random.default_rng(2)
    x0 = (rng.standard_normal((K, P)) * 0.02).astype(np.float32)
    starts = np.concatenate([[0], np.cumsum(numel)])
    whole = GpuRun(cfg, x0, numel=numel)
    parts = []
    for r in range(world):
        pieces = shard_ranges(numel, r, world, align=1024)
        ix = np.concatenate([np.arange(starts[j] + a, starts[j] + b) for j, a, b in pieces])
        parts.append((GpuRun(cfg, x0[:, ix], numel=[b - a for _, a, b in pieces]), ix))
    for t in range(cfg.T):
        g = np.stack([W.grads_host(P, cfg.grad_seed, t, k, cfg.grad_std) for k in range(K)])
        g = W.bf16_bits_from_f32_host(g) if precision else g
        whole.set_grads(g); whole.step(cfg.lr, cfg.eta)
        for run, ix in parts:
            run.set_grads(np.ascontiguousarray(g[:, ix])); run.step(cfg.lr, cfg.eta)
    sw = whole.state()
    for run, ix in parts:
        sp = run.state()
        for key in sp:
            want = sw[key][..., ix]
            assert np.array_equal(sp[key], want), key
        assert run.counters() == whole.counters()
