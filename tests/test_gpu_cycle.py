"""The captured synchronisation cycle (H inner steps + outer sync as one CUDA graph)
against step-by-step execution and against the CPU oracle."""
import numpy as np
import pytest

import paper_2504_18454_b200 as P
import workloads as W
from workloads.configs import WorkloadConfig
from _harness import GpuRun, compare_state, make_oracle

pytestmark = pytest.mark.gpu

RAGGED = [1, 3, 7, 1001, 4095, 4096, 4097, 0, 5, 12289, 8]


def _cfg(**kw):
    base = dict(name="cycle", shape=lambda: [], K=4, H=5, p=0.25, eta=16.0, lr=1e-3, T=15)
    base.update(kw)
    return WorkloadConfig(**base)


def _grads(cfg, Pn, t):
    g = np.stack([W.grads_host(Pn, cfg.grad_seed, t, k, cfg.grad_std) for k in range(cfg.K)])
    return W.bf16_bits_from_f32_host(g) if cfg.precision == 1 else g


def _x0(K, Pn, seed=1):
    return (np.random.default_rng(seed).standard_normal((K, Pn)) * 0.02).astype(np.float32)


@pytest.mark.parametrize("inner,precision,clip", [(0, 0, 0.0), (1, 0, 0.0), (0, 1, 0.0), (1, 1, 0.3), (0, 0, 0.3)])
def test_captured_cycle_equals_stepwise_execution_and_the_oracle(inner, precision, clip):
    cfg = _cfg(inner=inner, precision=precision, momentum=0.9 if inner else 0.0)
    Pn = sum(RAGGED)
    x0 = _x0(cfg.K, Pn)
    a, b, orc = GpuRun(cfg, x0, numel=RAGGED), GpuRun(cfg, x0, numel=RAGGED), make_oracle(cfg, x0)
    for r in (a, b, orc):
        r.set_grad_clip(clip)
    a.lib.cycle_capture(cfg.lr, cfg.eta)
    for cyc in range(3):
        g = _grads(cfg, Pn, cyc)                      # one gradient per cycle: the buffers stay as they are inside it
        a.set_grads(g); b.set_grads(g)
        a.lib.cycle_launch(a.stream)
        for _ in range(cfg.H):
            b.step(cfg.lr, cfg.eta); orc.step(g, cfg.lr, cfg.eta)
        sa, sb = a.state(), b.state()
        for key in sa:
            assert np.array_equal(sa[key], sb[key]), key
        assert a.counters() == b.counters()
    compare_state(a.state(), orc, exact=True)
    c = a.counters()
    assert c["t"] == 15 and c["n_outer"] == 3 and c["s"] == [int(v) for v in orc.s]
    assert a.lib.get_launch_count() == b.lib.get_launch_count()
    assert a.guards_intact()


def test_cycle_can_be_recaptured_with_new_rates_and_mixed_with_single_steps():
    numel = [9000, 5]
    cfg = _cfg(H=3)
    x0 = _x0(cfg.K, 9005)
    a, orc = GpuRun(cfg, x0, numel=numel), make_oracle(cfg, x0)
    g = _grads(cfg, 9005, 0)
    a.set_grads(g)
    for lr in (1e-3, 5e-4):
        a.lib.cycle_capture(lr, cfg.eta)
        a.lib.cycle_launch(a.stream)
        for _ in range(cfg.H):
            orc.step(g, lr, cfg.eta)
    for _ in range(cfg.H):                            # a cycle of single steps in between
        a.step(1e-3, cfg.eta); orc.step(g, 1e-3, cfg.eta)
    a.lib.cycle_launch(a.stream)                      # the recording (lr 5e-4) is still valid
    for _ in range(cfg.H):
        orc.step(g, 5e-4, cfg.eta)
    compare_state(a.state(), orc, exact=True)
    assert a.counters()["t"] == 12 and a.counters()["n_outer"] == 4


def test_cycle_state_errors():
    cfg = _cfg(H=4)
    r = GpuRun(cfg, _x0(cfg.K, 64), numel=[64])
    with pytest.raises(P.PalsgdError) as e:
        r.lib.cycle_launch(r.stream)                  # nothing recorded
    assert e.value.status == -4
    r.set_grads(_grads(cfg, 64, 0)); r.step(cfg.lr, cfg.eta)
    with pytest.raises(P.PalsgdError) as e:
        r.lib.cycle_capture(cfg.lr, cfg.eta)          # t = 1 is not the start of a cycle
    assert e.value.status == -4
    for _ in range(3):
        r.step(cfg.lr, cfg.eta)
    r.lib.cycle_capture(cfg.lr, cfg.eta)
    r.step(cfg.lr, cfg.eta)
    with pytest.raises(P.PalsgdError) as e:
        r.lib.cycle_launch(r.stream)                  # mid-cycle
    assert e.value.status == -4
    adam_outer = GpuRun(_cfg(outer_opt=1, outer_lr=0.01), _x0(4, 64), numel=[64])
    with pytest.raises(P.PalsgdError) as e:
        adam_outer.lib.cycle_capture(1e-3, 16.0)
    assert e.value.status == -6


def test_changing_a_launch_knob_drops_the_recorded_cycle():
    # the recording holds launch shapes and item-table addresses; a knob that rebuilds a table would leave
    # it pointing at freed memory, so any knob change invalidates it
    numel = [5000, 300]
    cfg = _cfg(H=2)
    x0 = _x0(cfg.K, 5300)
    a, orc = GpuRun(cfg, x0, numel=numel), make_oracle(cfg, x0)
    g = _grads(cfg, 5300, 0)
    a.set_grads(g)
    a.lib.cycle_capture(cfg.lr, cfg.eta)
    a.lib.cycle_launch(a.stream)
    a.lib.set_tuning(P.TUNE_OUTER_SUB_ELEMS, 2048)
    with pytest.raises(P.PalsgdError) as e:
        a.lib.cycle_launch(a.stream)
    assert e.value.status == -4
    a.lib.cycle_capture(cfg.lr, cfg.eta)              # recorded again with the new table
    a.lib.cycle_launch(a.stream)
    for _ in range(2 * cfg.H):
        orc.step(g, cfg.lr, cfg.eta)
    compare_state(a.state(), orc, exact=True)
