"""The outer synchronisation with the K workers spread over several contexts (one per GPU in a
real deployment): palsgd_outer_partial -> sum of the exchange buffers -> palsgd_outer_finish.

One GPU is at hand, so the several-rank case runs as several contexts on that GPU, one launch
after the other (nothing waits on anything), with a plain tensor addition standing in for the
all-reduce between two ranks (one commutative addition, so the result is the collective's).
"""
import numpy as np
import pytest
import torch

import workloads as W
from workloads.configs import WorkloadConfig
from paper_2504_18454_b200.workers import DistributedPalsgd
from _harness import GpuRun, compare_state, make_oracle

pytestmark = pytest.mark.gpu

RAGGED = [4096 * 3 + 5, 7, 1001, 0, 8192, 12]


def _cfg(**kw):
    base = dict(name="workers", shape=lambda: [], K=4, H=3, p=0.3, eta=16.0, lr=1e-3, T=7)
    base.update(kw)
    return WorkloadConfig(**base)


def _grads(cfg, P, t, K_total):
    g = np.stack([W.grads_host(P, cfg.grad_seed, t, k, cfg.grad_std) for k in range(K_total)])
    return W.bf16_bits_from_f32_host(g) if cfg.precision == 1 else g


@pytest.mark.parametrize("layout", ["arena", "separate", "misaligned"])
@pytest.mark.parametrize("precision,outer_opt", [(0, 0), (1, 0), (0, 1), (1, 1)])
def test_one_rank_is_bit_identical_to_the_plain_outer_sync(layout, precision, outer_opt):
    cfg = _cfg(precision=precision, outer_opt=outer_opt, outer_lr=0.7 if outer_opt == 0 else 0.02)
    P = sum(RAGGED)
    rng = np.random.default_rng(3)
    x0 = (rng.standard_normal((cfg.K, P)) * 0.02).astype(np.float32)
    plain, orc = GpuRun(cfg, x0, numel=RAGGED, layout=layout), make_oracle(cfg, x0)
    split = GpuRun(cfg, x0, numel=RAGGED, layout=layout)
    exch = torch.zeros(split.lib.exchange_numel(), dtype=torch.float32, device=split.dev)
    assert exch.numel() >= P
    job = DistributedPalsgd(split.lib, exch, cfg.K, 0, 1, all_reduce_sum=lambda buf: None)
    job.init_global(split.stream)                              # one rank: the mean palsgd_init formed, bit for bit
    assert np.array_equal(split.state()["xg"], plain.state()["xg"])
    for t in range(cfg.T):
        g = _grads(cfg, P, t, cfg.K)
        plain.set_grads(g); split.set_grads(g)
        plain.step(cfg.lr, cfg.eta); orc.step(g, cfg.lr, cfg.eta)
        assert job.step(cfg.lr, cfg.eta, split.stream) == ((t + 1) % cfg.H == 0)
    a, b = plain.state(), split.state()
    for key in a:
        assert np.array_equal(a[key], b[key]), key
    compare_state(b, orc, exact=True)
    assert split.counters()["n_outer"] == cfg.T // cfg.H and split.guards_intact()


@pytest.mark.parametrize("inner,precision", [(0, 0), (1, 0), (0, 1)])
def test_two_ranks_with_half_of_the_workers_each_match_the_oracle_bit_for_bit(inner, precision):
    K_total, world = 6, 2
    cfg = _cfg(K=K_total, inner=inner, precision=precision, momentum=0.9 if inner else 0.0, p=0.35)
    P = sum(RAGGED)
    x0 = (np.random.default_rng(9).standard_normal((K_total, P)) * 0.02).astype(np.float32)   # workers start apart
    from _harness import cfg_kwargs
    import oracle
    orc = oracle.Oracle(x0, sum_groups=world, **cfg_kwargs(cfg))     # sums per rank first, then across the two ranks
    local = cfg.with_(K=K_total // world)
    ranks = [GpuRun(local, x0[r * local.K:(r + 1) * local.K], numel=RAGGED, layout="separate" if r else "arena")
             for r in range(world)]
    for r, run in enumerate(ranks):
        run.lib.set_worker_offset(r * local.K)
    exch = [torch.zeros(run.lib.exchange_numel(), dtype=torch.float32, device=run.dev) for run in ranks]
    # the job's initial global model: the mean over all workers, formed through the same exchange
    for run, e in zip(ranks, exch):
        run.lib.outer_partial(e.data_ptr(), run.stream)
    total = exch[0] + exch[1]
    for run, e in zip(ranks, exch):
        e.copy_(total)
        run.lib.global_from_exchange(e.data_ptr(), K_total, run.stream)
        assert np.array_equal(run.state()["xg"], orc.xg)
    for t in range(cfg.T):
        g = _grads(cfg, P, t, K_total)
        orc.step(g, cfg.lr, cfg.eta)
        for r, run in enumerate(ranks):
            run.set_grads(g[r * local.K:(r + 1) * local.K])
            run.inner_step(cfg.lr, cfg.eta)
            c = run.counters()                                  # the job's decisions, bit for bit
            assert c["last_b"] == [int(v) for v in orc.last_b[r * local.K:(r + 1) * local.K]]
        if (t + 1) % cfg.H == 0:
            for run, e in zip(ranks, exch):
                run.lib.outer_partial(e.data_ptr(), run.stream)
            total = exch[0] + exch[1]                           # the all-reduce of two ranks: one addition
            for run, e in zip(ranks, exch):
                e.copy_(total)
                run.lib.outer_finish(e.data_ptr(), K_total, run.stream)
    states = [run.state() for run in ranks]
    assert any(int(v) < cfg.T for v in orc.s) and orc.n_outer == 2
    for key in ("xg", "u"):                                     # every rank holds the same global model
        assert np.array_equal(states[0][key], states[1][key]), key
    for r, (run, st) in enumerate(zip(ranks, states)):
        sl = slice(r * local.K, (r + 1) * local.K)
        assert run.counters()["s"] == [int(v) for v in orc.s[sl]]

        class View:                                             # the oracle's rows of this rank
            dtype = orc.dtype
            x, m, v, xg, u, uv = orc.x[sl], orc.m[sl], orc.v[sl], orc.xg, orc.u, None
            xw = orc.xw[sl] if orc.xw is not None else None
        # the oracle adds the two ranks' partial sums exactly as the exchange does (two groups), so the
        # comparison is bit for bit; against the one-level ascending sum only the parity bar would hold
        compare_state(st, View, exact=True)
        assert run.guards_intact()


@pytest.mark.parametrize("layout", ["arena", "separate", "misaligned"])
@pytest.mark.parametrize("inner,precision", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_one_rank_ddp_step_through_the_exchange_is_bit_identical_to_the_plain_one(layout, inner, precision):
    cfg = _cfg(inner=inner, precision=precision, momentum=0.9 if inner else 0.0)
    P = sum(RAGGED)
    x0 = np.tile((np.random.default_rng(5).standard_normal(P) * 0.02).astype(np.float32), (cfg.K, 1))
    plain, split, orc = (GpuRun(cfg, x0, numel=RAGGED, layout=layout), GpuRun(cfg, x0, numel=RAGGED, layout=layout),
                         make_oracle(cfg, x0))
    exch = torch.zeros(split.lib.exchange_numel(), dtype=torch.float32, device=split.dev)
    job = DistributedPalsgd(split.lib, exch, cfg.K, 0, 1, all_reduce_sum=lambda buf: None)
    for t in range(4):
        g = _grads(cfg, P, t, cfg.K)
        plain.set_grads(g); split.set_grads(g)
        plain.ddp_step(cfg.lr); job.ddp_step(cfg.lr, split.stream); orc.ddp_step(g, cfg.lr)
    a, b = plain.state(), split.state()
    for key in a:
        assert np.array_equal(a[key], b[key]), key
    compare_state(b, orc, exact=True)
    assert split.counters()["t"] == 4 and split.counters()["s"] == [4] * cfg.K and split.guards_intact()
    for t in range(4, 4 + cfg.T):                                # and on into Algorithm 1 from that state
        g = _grads(cfg, P, t, cfg.K)
        split.set_grads(g); orc.step(g, cfg.lr, cfg.eta); job.step(cfg.lr, cfg.eta, split.stream)
    compare_state(split.state(), orc, exact=True)


@pytest.mark.parametrize("inner,precision", [(0, 0), (1, 0), (0, 1), (1, 1)])
def test_two_ranks_ddp_warm_up_then_algorithm_1_match_the_oracle_bit_for_bit(inner, precision):
    K_total, world, n_ddp = 6, 2, 3
    cfg = _cfg(K=K_total, inner=inner, precision=precision, momentum=0.9 if inner else 0.0, p=0.35, T=6)
    P = sum(RAGGED)
    x0 = np.tile((np.random.default_rng(11).standard_normal(P) * 0.02).astype(np.float32), (K_total, 1))
    from _harness import cfg_kwargs
    import oracle
    orc = oracle.Oracle(x0, sum_groups=world, **cfg_kwargs(cfg))
    local = cfg.with_(K=K_total // world)
    ranks = [GpuRun(local, x0[r * local.K:(r + 1) * local.K], numel=RAGGED, layout="misaligned" if r else "arena", row_align=256 if r else 8)
             for r in range(world)]
    exch = [torch.zeros(run.lib.exchange_numel(), dtype=torch.float32, device=run.dev) for run in ranks]

    def exchange_sum():                                         # the all-reduce of two ranks: one addition
        total = exch[0] + exch[1]
        for e in exch:
            e.copy_(total)

    for r, run in enumerate(ranks):
        run.lib.set_worker_offset(r * local.K)
    for t in range(n_ddp):
        g = _grads(cfg, P, t, K_total)
        orc.ddp_step(g, cfg.lr)
        for r, run in enumerate(ranks):
            run.set_grads(g[r * local.K:(r + 1) * local.K])
            run.lib.ddp_partial(exch[r].data_ptr(), run.stream)
        exchange_sum()
        for r, run in enumerate(ranks):
            run.lib.ddp_finish(exch[r].data_ptr(), K_total, cfg.lr, run.stream)
    states = [run.state() for run in ranks]
    for key in ("x", "m", "xg"):                                # all ranks took the same step
        assert np.array_equal(states[0][key], states[1][key]), key
    assert np.array_equal(states[0]["xg"], orc.xg) and np.array_equal(states[0]["x"][0], orc.x[0])
    for t in range(n_ddp, n_ddp + cfg.T):
        g = _grads(cfg, P, t, K_total)
        orc.step(g, cfg.lr, cfg.eta)
        for r, run in enumerate(ranks):
            run.set_grads(g[r * local.K:(r + 1) * local.K])
            run.inner_step(cfg.lr, cfg.eta)
        if (t + 1) % cfg.H == 0:
            for r, run in enumerate(ranks):
                run.lib.outer_partial(exch[r].data_ptr(), run.stream)
            exchange_sum()
            for r, run in enumerate(ranks):
                run.lib.outer_finish(exch[r].data_ptr(), K_total, run.stream)
    assert orc.n_outer >= 2
    for r, run in enumerate(ranks):
        sl = slice(r * local.K, (r + 1) * local.K)
        assert run.counters()["s"] == [int(v) for v in orc.s[sl]] and run.counters()["t"] == orc.t

        class View:
            dtype = orc.dtype
            x, m, v, xg, u, uv = orc.x[sl], orc.m[sl], orc.v[sl], orc.xg, orc.u, None
            xw = orc.xw[sl] if orc.xw is not None else None
        compare_state(run.state(), View, exact=True)
        assert run.guards_intact()


def test_argument_checks():
    cfg = _cfg()
    run = GpuRun(cfg, np.zeros((cfg.K, 100), dtype=np.float32), numel=[100])
    buf = torch.zeros(run.lib.exchange_numel() + 4, dtype=torch.float32, device=run.dev)
    for call in (lambda: run.lib.outer_partial(0, run.stream), lambda: run.lib.outer_finish(0, cfg.K, run.stream),
                 lambda: run.lib.outer_finish(buf.data_ptr(), cfg.K - 1, run.stream),
                 lambda: run.lib.global_from_exchange(0, cfg.K, run.stream),
                 lambda: run.lib.global_from_exchange(buf.data_ptr(), cfg.K - 1, run.stream)):
        with pytest.raises(Exception) as e:
            call()
        assert getattr(e.value, "status", None) == -1
    with pytest.raises(Exception) as e:
        run.lib.outer_partial(buf.data_ptr() + 4, run.stream)
    assert getattr(e.value, "status", None) == -2
    for call in (lambda: run.lib.ddp_partial(0, run.stream), lambda: run.lib.ddp_finish(0, cfg.K, 1e-3, run.stream),
                 lambda: run.lib.ddp_finish(buf.data_ptr(), cfg.K - 1, 1e-3, run.stream),
                 lambda: run.lib.ddp_finish(buf.data_ptr(), cfg.K, float("nan"), run.stream)):
        with pytest.raises(Exception) as e:
            call()
        assert getattr(e.value, "status", None) == -1
    with pytest.raises(Exception) as e:
        run.lib.ddp_partial(buf.data_ptr() + 4, run.stream)
    assert getattr(e.value, "status", None) == -2
    run.set_grad_clip(1.0)                                       # no clipped form of the split step
    run.lib.ddp_partial(buf.data_ptr(), run.stream)
    with pytest.raises(Exception) as e:
        run.lib.ddp_finish(buf.data_ptr(), cfg.K, 1e-3, run.stream)
    assert getattr(e.value, "status", None) == -6
    c = run.counters()
    assert c["n_outer"] == 0 and c["t"] == 0
