"""GPU parity of the DDP warm-up step (the mini-batch phase that precedes
Algorithm 1) against the CPU oracle, element by element: ragged tensor lists,
both optimizers, both precisions, all buffer layouts, the switch into the
PALSGD phase, and resume."""
import numpy as np
import pytest

import workloads as W
from workloads.configs import WorkloadConfig
from _harness import GpuRun, compare_state, make_oracle

pytestmark = pytest.mark.gpu

RAGGED = [1, 3, 7, 1001, 4095, 4096, 4097, 0, 5, 12289, 8]


def _cfg(**kw):
    base = dict(name="ddp", shape=lambda: [], K=4, H=4, p=0.25, eta=16.0, lr=1e-3, T=10)
    base.update(kw)
    return WorkloadConfig(**base)


def _grads(cfg, P, t):
    g = np.stack([W.grads_host(P, cfg.grad_seed, t, k, cfg.grad_std) for k in range(cfg.K)])
    return W.bf16_bits_from_f32_host(g) if cfg.precision == 1 else g


def _x0(K, P, seed=1, same=True):
    rng = np.random.default_rng(seed)
    if same:
        return np.tile((rng.standard_normal(P) * 0.02).astype(np.float32), (K, 1))
    return (rng.standard_normal((K, P)) * 0.02).astype(np.float32)


def _warmup_then_palsgd(cfg, numel, layout, n_ddp, n_palsgd, x0=None):
    P = int(sum(numel))
    x0 = _x0(cfg.K, P) if x0 is None else x0
    gpu, orc = GpuRun(cfg, x0, numel=numel, layout=layout), make_oracle(cfg, x0)
    for t in range(n_ddp):
        g = _grads(cfg, P, t)
        gpu.set_grads(g); gpu.ddp_step(cfg.lr); orc.ddp_step(g, cfg.lr)
        c = gpu.counters()
        assert c["t"] == orc.t and c["s"] == [int(v) for v in orc.s] and c["last_b"] == [0] * cfg.K
    st = gpu.state()
    compare_state(st, orc, exact=True)
    for k in range(cfg.K):                                        # the DDP invariant, bitwise
        assert np.array_equal(st["x"][k], st["xg"]) and np.array_equal(st["m"][k], st["m"][0])
    for t in range(n_ddp, n_ddp + n_palsgd):
        g = _grads(cfg, P, t)
        gpu.set_grads(g); gpu.step(cfg.lr, cfg.eta); orc.step(g, cfg.lr, cfg.eta)
        c = gpu.counters()
        assert c["last_b"] == [int(v) for v in orc.last_b] and c["s"] == [int(v) for v in orc.s]
    compare_state(gpu.state(), orc, exact=True)
    c = gpu.counters()
    assert c["t"] == orc.t == n_ddp + n_palsgd and c["n_outer"] == orc.n_outer
    assert gpu.guards_intact()
    return gpu, orc


@pytest.mark.parametrize("layout", ["arena", "separate", "misaligned"])
@pytest.mark.parametrize("inner,precision", [(0, 0), (1, 0), (0, 1), (1, 1)])
def test_ragged_list_warm_up_then_palsgd(layout, inner, precision):
    cfg = _cfg(inner=inner, precision=precision, momentum=0.9 if inner else 0.0,
               weight_decay=1e-4 if inner else 0.01)
    _warmup_then_palsgd(cfg, RAGGED, layout, n_ddp=5, n_palsgd=7)


@pytest.mark.parametrize("K", [1, 2, 3, 8, 17, 64])
def test_worker_counts(K):
    numel = [4096 * 2 + 13]
    _warmup_then_palsgd(_cfg(K=K, H=3), numel, "arena", n_ddp=3, n_palsgd=4)
    _warmup_then_palsgd(_cfg(K=K, H=3, precision=1), numel, "arena", n_ddp=2, n_palsgd=2)


@pytest.mark.parametrize("numel", [[1], [3], [4095], [0, 0, 2]])
def test_tiny_sizes(numel):
    _warmup_then_palsgd(_cfg(K=3, H=2), numel, "separate", n_ddp=3, n_palsgd=3)


def test_slots_that_differ_follow_worker_zero():
    numel = [6000, 11]
    _warmup_then_palsgd(_cfg(K=5), numel, "arena", n_ddp=2, n_palsgd=0, x0=_x0(5, 6011, seed=4, same=False))


def test_launch_shape_independence_and_launch_count():
    numel = RAGGED
    P = sum(numel)
    cfg = _cfg(K=8)
    outs = []
    for cap in (0, 3, 148):
        r = GpuRun(cfg, _x0(8, P), numel=numel)
        r.lib.set_tuning(1, cap)
        for t in range(4):
            r.set_grads(_grads(cfg, P, t)); r.ddp_step(cfg.lr)
        outs.append(r.state())
        assert r.lib.get_launch_count() == 1 + 4                  # init + one launch per step
    for o in outs[1:]:
        for k in outs[0]:
            assert np.array_equal(outs[0][k], o[k]), k


@pytest.mark.parametrize("inner,precision", [(0, 0), (1, 0), (0, 1), (1, 1)])
@pytest.mark.parametrize("variant,sub,dyn", [(1, 1024, 0), (2, 1024, 0), (2, 2048, 0), (2, 3072, 0), (2, 8192, 0),
                                             (1, 1024, 3), (2, 2048, 2)])
def test_every_form_of_the_ddp_kernel_matches_oracle(variant, sub, dyn, inner, precision):
    # variant 2 stages the new state in shared memory and writes the K slots with bulk asynchronous
    # stores; slices that do not fit the stage fall back to per-thread stores
    numel = [4096 * 5 + 4, 12, 8192 + 6, 1001]
    P = sum(numel)
    cfg = _cfg(K=5, inner=inner, precision=precision, momentum=0.9 if inner else 0.0)
    for layout, cap in (("arena", 0), ("separate", 3), ("misaligned", 0)):
        x0 = _x0(cfg.K, P, seed=8)
        gpu, orc = GpuRun(cfg, x0, numel=numel, layout=layout), make_oracle(cfg, x0)
        gpu.lib.set_tuning(7, variant); gpu.lib.set_tuning(6, sub); gpu.lib.set_tuning(1, cap)
        gpu.lib.set_tuning(9, dyn)                    # persistent grid + work queue (ignored when the grid is capped)
        for t in range(4):
            g = _grads(cfg, P, t)
            gpu.set_grads(g); gpu.ddp_step(cfg.lr); orc.ddp_step(g, cfg.lr)
        compare_state(gpu.state(), orc, exact=True)
        assert gpu.guards_intact()


def test_resume_inside_the_warm_up_is_bit_exact():
    numel = [10000]
    cfg = _cfg()
    x0 = _x0(cfg.K, 10000)
    a = GpuRun(cfg, x0, numel=numel)
    for t in range(6):
        a.set_grads(_grads(cfg, 10000, t)); a.ddp_step(cfg.lr)
    b = GpuRun(cfg, x0, numel=numel)
    for t in range(3):
        b.set_grads(_grads(cfg, 10000, t)); b.ddp_step(cfg.lr)
    saved, cnt = b.state(), b.counters()
    c = GpuRun(cfg, x0, numel=numel)
    for name, key in (("param", "x"), ("m", "m"), ("v", "v")):
        c._write(name, saved[key])
    c._write("global_", saved["xg"][None]); c._write("outer_mom", saved["u"][None])
    c.lib.set_counters(cnt["t"], cnt["s"], cnt["n_outer"], c.stream)
    for t in range(3, 6):
        c.set_grads(_grads(cfg, 10000, t)); c.ddp_step(cfg.lr)
    want, got = a.state(), c.state()
    for k in want:
        assert np.array_equal(want[k], got[k]), k
    assert c.counters() == a.counters()


def test_bad_arguments():
    cfg = _cfg()
    r = GpuRun(cfg, _x0(cfg.K, 64), numel=[64])
    for bad in (-1.0, float("nan"), float("inf")):
        with pytest.raises(Exception):
            r.ddp_step(bad)
