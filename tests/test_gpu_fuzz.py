"""Seeded random sweep over tensor lists, worker counts, precisions, optimizers, device layouts and
launch-shape knobs: a DDP warm-up step or two, then Algorithm 1 with clipping and outer syncs,
compared with the oracle bit for bit.  The shapes are drawn around the sizes where the kernels
change path: 4 / 8-element groups, 1024-element items, 4096 / 8192-element chunks, empty tensors."""
import numpy as np
import pytest

import paper_2504_18454_b200 as P
import workloads as W
from workloads.configs import WorkloadConfig
from _harness import GpuRun, compare_state, make_oracle

pytestmark = pytest.mark.gpu

EDGES = [0, 1, 3, 4, 5, 7, 8, 9, 15, 16, 17, 255, 256, 1023, 1024, 1025, 2047, 2048, 4095, 4096, 4097,
         8191, 8192, 8193, 12288, 16385]


def _case(seed):
    rng = np.random.default_rng(1000 + seed)
    n = int(rng.integers(1, 7))
    numel = [int(rng.choice(EDGES)) + int(rng.integers(0, 2)) * int(rng.integers(0, 40)) for _ in range(n)]
    if sum(numel) == 0:
        numel[0] = 33
    K = int(rng.choice([1, 2, 3, 4, 5, 8, 9, 17]))
    inner = int(rng.integers(0, 2))
    cfg = WorkloadConfig(name=f"fuzz{seed}", shape=lambda: [], K=K, H=int(rng.choice([1, 2, 3])),
                         p=float(rng.choice([0.0, 0.3, 0.5, 1.0])), eta=16.0, lr=1e-3, T=5,
                         inner=inner, momentum=0.9 if inner else 0.0, precision=int(rng.integers(0, 2)),
                         outer_opt=int(rng.integers(0, 2)) if rng.random() < 0.3 else 0,
                         outer_lr=0.7, outer_nesterov=bool(rng.integers(0, 2)))
    if cfg.outer_opt == 1:
        cfg = cfg.with_(outer_lr=0.02)
    layout = str(rng.choice(["arena", "separate", "misaligned"]))
    knobs = {}
    if rng.random() < 0.6:
        knobs[P.TUNE_OUTER_SUB_ELEMS] = int(rng.choice([1024, 2048, 4096]))
        knobs[P.TUNE_DDP_SUB_ELEMS] = int(rng.choice([1024, 2048, 3072]))
        knobs[P.TUNE_OUTER_DYNAMIC] = int(rng.choice([0, 1, 3]))
        knobs[P.TUNE_OUTER_GRID_CAP] = int(rng.choice([0, 0, 2, 5]))
        knobs[P.TUNE_INNER_GRID_CAP] = int(rng.choice([0, 0, 3]))
        knobs[P.TUNE_INNER_VARIANT] = int(rng.choice([0, 18]))
        knobs[P.TUNE_OUTER_VARIANT] = int(rng.choice([0, 1, 2]))
        knobs[P.TUNE_DDP_VARIANT] = int(rng.choice([0, 1, 2]))
    n_ddp = int(rng.integers(0, 3))
    clip = float(rng.choice([0.0, 0.0, 0.05]))
    # where the rows of a packed layout start: how far apart (elements) and how far off that grid; decides the
    # scalar head the library peels (0 to 255 elements)
    place = np.random.default_rng(5000 + seed)
    geometry = dict(row_align=int(place.choice([8, 8, 64, 128, 256])), shift=int(place.choice([1, 1, 2, 3, 5, 100, 201])))
    return cfg, numel, layout, knobs, n_ddp, clip, geometry


@pytest.mark.parametrize("seed", range(160))
def test_random_configuration_matches_the_oracle_bit_for_bit(seed):
    cfg, numel, layout, knobs, n_ddp, clip, geometry = _case(seed)
    Pn = int(sum(numel))
    x0 = (np.random.default_rng(seed).standard_normal((cfg.K, Pn)) * 0.02).astype(np.float32)
    if n_ddp:
        x0 = np.tile(x0[0], (cfg.K, 1))                  # the warm-up phase starts from a common model
    gpu, orc = GpuRun(cfg, x0, numel=numel, layout=layout, **geometry), make_oracle(cfg, x0)
    for knob, value in knobs.items():
        gpu.lib.set_tuning(knob, value)
    if clip:
        gpu.set_grad_clip(clip); orc.set_grad_clip(clip)
    for t in range(n_ddp + cfg.T):
        g = np.stack([W.grads_host(Pn, cfg.grad_seed, t, k, cfg.grad_std) for k in range(cfg.K)])
        g = W.bf16_bits_from_f32_host(g) if cfg.precision == 1 else g
        gpu.set_grads(g)
        if t < n_ddp:
            gpu.ddp_step(cfg.lr); orc.ddp_step(g, cfg.lr)
        else:
            gpu.step(cfg.lr, cfg.eta); orc.step(g, cfg.lr, cfg.eta)
    compare_state(gpu.state(), orc, exact=True)
    c = gpu.counters()
    assert c["t"] == orc.t and c["n_outer"] == orc.n_outer and c["s"] == [int(v) for v in orc.s]
    assert c["last_b"] == [int(v) for v in orc.last_b] and gpu.guards_intact()
