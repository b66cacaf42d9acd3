"""GPU parity of the outer-optimizer variants (AdamW as OuterOPT, a scheduled outer
learning rate) against the CPU oracle, and the host schedule function against the
oracle's."""
import numpy as np
import pytest

import oracle
import paper_2504_18454_b200 as P
import workloads as W
from workloads.configs import WorkloadConfig
from _harness import GpuRun, compare_state, make_oracle

RAGGED = [1, 3, 7, 1001, 4095, 4096, 4097, 0, 5, 12289, 8]


def _cfg(**kw):
    base = dict(name="ov", shape=lambda: [], K=4, H=3, p=0.25, eta=16.0, lr=1e-3, T=10)
    base.update(kw)
    return WorkloadConfig(**base)


def _grads(cfg, Pn, t):
    g = np.stack([W.grads_host(Pn, cfg.grad_seed, t, k, cfg.grad_std) for k in range(cfg.K)])
    return W.bf16_bits_from_f32_host(g) if cfg.precision == 1 else g


def _x0(K, Pn, seed=1):
    return (np.random.default_rng(seed).standard_normal((K, Pn)) * 0.02).astype(np.float32)


@pytest.mark.gpu
@pytest.mark.parametrize("layout", ["arena", "separate", "misaligned"])
@pytest.mark.parametrize("precision", [0, 1])
def test_adamw_outer_matches_oracle(layout, precision):
    cfg = _cfg(precision=precision, outer_opt=1, outer_lr=0.01, outer_beta2=0.95, outer_weight_decay=0.05)
    Pn = sum(RAGGED)
    x0 = _x0(cfg.K, Pn)
    gpu, orc = GpuRun(cfg, x0, numel=RAGGED, layout=layout), make_oracle(cfg, x0)
    for t in range(cfg.T):
        g = _grads(cfg, Pn, t)
        gpu.set_grads(g); gpu.step(cfg.lr, cfg.eta); orc.step(g, cfg.lr, cfg.eta)
    st = gpu.state()
    compare_state(st, orc, exact=True)
    assert "uv" in st and np.any(st["uv"] != 0)
    assert gpu.counters()["n_outer"] == orc.n_outer == 3 and gpu.guards_intact()


@pytest.mark.gpu
@pytest.mark.parametrize("K", [1, 3, 9, 64])
def test_adamw_outer_worker_counts_and_inner_sgd(K):
    numel = [4096 * 3 + 5, 9]
    cfg = _cfg(K=K, H=2, T=6, inner=1, momentum=0.9, outer_opt=1, outer_lr=0.02)
    x0 = _x0(K, sum(numel))
    gpu, orc = GpuRun(cfg, x0, numel=numel), make_oracle(cfg, x0)
    for t in range(cfg.T):
        g = _grads(cfg, sum(numel), t)
        gpu.set_grads(g); gpu.step(cfg.lr, cfg.eta); orc.step(g, cfg.lr, cfg.eta)
    compare_state(gpu.state(), orc, exact=True)


@pytest.mark.gpu
@pytest.mark.parametrize("outer_opt", [0, 1])
def test_scheduled_outer_learning_rate(outer_opt):
    numel = [9000, 77]
    Pn = sum(numel)
    cfg = _cfg(H=2, T=12, outer_opt=outer_opt, outer_lr=0.7 if outer_opt == 0 else 0.02)
    x0 = _x0(cfg.K, Pn)
    gpu, orc = GpuRun(cfg, x0, numel=numel), make_oracle(cfg, x0)
    for t in range(cfg.T):
        rnd = t // cfg.H
        lr_lib = P.schedule_value(P.SCHED_WARMUP_COSINE, rnd, 2, 6, cfg.outer_lr, 0.01 * cfg.outer_lr, 0.1)
        lr_orc = oracle.schedule(1, rnd, 2, 6, cfg.outer_lr, 0.01 * cfg.outer_lr, 0.1)
        assert lr_lib == lr_orc
        gpu.set_outer_lr(lr_lib); orc.set_outer_lr(lr_orc)
        g = _grads(cfg, Pn, t)
        gpu.set_grads(g); gpu.step(cfg.lr, cfg.eta); orc.step(g, cfg.lr, cfg.eta)
    compare_state(gpu.state(), orc, exact=True)


@pytest.mark.gpu
def test_adamw_outer_resume_restores_the_outer_step_count():
    numel = [10000]
    cfg = _cfg(H=2, outer_opt=1, outer_lr=0.01)
    x0 = _x0(cfg.K, 10000)
    a = GpuRun(cfg, x0, numel=numel)
    for t in range(8):
        a.set_grads(_grads(cfg, 10000, t)); a.step(cfg.lr, cfg.eta)
    b = GpuRun(cfg, x0, numel=numel)
    for t in range(4):
        b.set_grads(_grads(cfg, 10000, t)); b.step(cfg.lr, cfg.eta)
    saved, cnt = b.state(), b.counters()
    c = GpuRun(cfg, x0, numel=numel)
    for name, key in (("param", "x"), ("m", "m"), ("v", "v")):
        c._write(name, saved[key])
    c._write("global_", saved["xg"][None]); c._write("outer_mom", saved["u"][None]); c._write("outer_v", saved["uv"][None])
    c.lib.set_counters(cnt["t"], cnt["s"], cnt["n_outer"], c.stream)
    for t in range(4, 8):
        c.set_grads(_grads(cfg, 10000, t)); c.step(cfg.lr, cfg.eta)
    want, got = a.state(), c.state()
    for k in want:
        assert np.array_equal(want[k], got[k]), k


@pytest.mark.gpu
def test_adamw_outer_needs_its_second_moment_buffer():
    import torch
    dev = torch.device("cuda:0")
    t = lambda: [[torch.zeros(16, device=dev)]]
    with pytest.raises(P.PalsgdError) as e:
        P.Palsgd(K=1, H=1, p=0.0, numel=[16], params=t(), grads=t(), m=t(), v=t(), global_=t()[0],
                 outer_mom=t()[0], outer_opt=P.OUTER_ADAMW)
    assert e.value.status == -1


def test_schedule_value_equals_the_oracle_schedule_on_a_grid():
    for kind in (0, 1):
        for warmup, total in ((0, 10), (5, 50), (10, 10), (7, 1000)):
            for t in list(range(0, 60)) + [999, 1000, 5000]:
                for sf, mn in ((0.0, 0.0), (0.1, 0.02), (1.0, 0.5)):
                    assert P.schedule_value(kind, t, warmup, total, 0.8, mn, sf) == \
                        oracle.schedule(kind, t, warmup, total, 0.8, mn, sf)


def test_schedule_value_rejects_bad_arguments():
    assert np.isnan(P.schedule_value(7, 0, 1, 2, 1.0))
    assert np.isnan(P.schedule_value(0, 0, 1, 2, float("inf")))


@pytest.mark.gpu
@pytest.mark.parametrize("precision,outer_opt", [(0, 0), (1, 0), (0, 1), (1, 1)])
@pytest.mark.parametrize("variant,sub,dyn", [(1, 1024, 0), (2, 1024, 0), (2, 2048, 0), (2, 4096, 0), (2, 16384, 0),
                                             (1, 1024, 2), (2, 1024, 4), (2, 4096, 1)])
def test_every_form_of_the_outer_kernel_matches_oracle(variant, sub, dyn, precision, outer_opt):
    # variant 2 stages the new global model in shared memory and writes the K slots with bulk
    # asynchronous stores; odd tails and unaligned segments take the per-thread stores
    numel = [4096 * 5 + 4, 12, 8192 + 6, 1001]
    Pn = sum(numel)
    cfg = _cfg(K=5, H=2, T=6, precision=precision, outer_opt=outer_opt, outer_lr=0.7 if outer_opt == 0 else 0.02)
    for layout, cap in (("arena", 0), ("separate", 3), ("misaligned", 0)):
        x0 = _x0(cfg.K, Pn, seed=8)
        gpu, orc = GpuRun(cfg, x0, numel=numel, layout=layout), make_oracle(cfg, x0)
        gpu.lib.set_tuning(8, variant); gpu.lib.set_tuning(5, sub); gpu.lib.set_tuning(1, cap)
        gpu.lib.set_tuning(9, dyn)                    # persistent grid + work queue (ignored when the grid is capped)
        for t in range(cfg.T):
            g = _grads(cfg, Pn, t)
            gpu.set_grads(g); gpu.step(cfg.lr, cfg.eta); orc.step(g, cfg.lr, cfg.eta)
        compare_state(gpu.state(), orc, exact=True)
        assert gpu.guards_intact()


@pytest.mark.gpu
def test_two_contexts_with_different_item_sizes_do_not_lower_each_others_shared_memory_limit():
    # the dynamic-shared-memory limit belongs to the kernel on the device: the context with the larger
    # stage sets it first, the one with the smaller stage must not lower it
    numel = [16384 * 2 + 40]
    Pn = sum(numel)
    cfg = _cfg(K=3, H=1, T=3)
    x0 = _x0(cfg.K, Pn, seed=4)
    big, small, orc = GpuRun(cfg, x0, numel=numel), GpuRun(cfg, x0, numel=numel), make_oracle(cfg, x0)
    big.lib.set_tuning(5, 16384)          # 128 KB of stage per CTA
    small.lib.set_tuning(5, 8192)         # 64 KB
    for t in range(cfg.T):
        g = _grads(cfg, Pn, t)
        orc.step(g, cfg.lr, cfg.eta)
        big.set_grads(g); small.set_grads(g)
        big.step(cfg.lr, cfg.eta); small.step(cfg.lr, cfg.eta)      # H = 1: big, small, big, small, ... outer syncs
    compare_state(big.state(), orc, exact=True)
    compare_state(small.state(), orc, exact=True)
