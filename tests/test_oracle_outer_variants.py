"""Pins for the outer-optimizer variants of the paper's optimizer ablation
(Appendix D: SGD, SGD with momentum, Nesterov, AdamW as OuterOPT) and for the
learning-rate schedule of Appendix B (warm-up, then cosine annealing)."""
import math

import numpy as np
import pytest
import torch

import oracle

RNG = np.random.default_rng(23)


def _mk(K, P, dtype="f64", **kw):
    x0 = (RNG.standard_normal((K, P)) * 0.02).astype(np.float32)
    cfg = dict(K=K, H=1, p=0.0, inner=1, momentum=0.0, weight_decay=0.0, seed=3)
    cfg.update(kw)
    return x0, oracle.Oracle(x0, dtype=dtype, **cfg)


@pytest.mark.parametrize("wd", [0.0, 0.05])
def test_adamw_outer_matches_torch_adamw_fed_the_outer_gradient(wd):
    # drive the local models by hand, take Delta = x - mean_k x_k, feed it to the library optimizer
    K, P, rounds = 3, 97, 12
    x0, o = _mk(K, P, outer_opt=1, outer_lr=0.01, outer_beta1=0.9, outer_beta2=0.95, outer_eps=1e-8,
                outer_weight_decay=wd)
    q = torch.tensor(o.xg.astype(np.float64).copy(), requires_grad=True)
    opt = torch.optim.AdamW([q], lr=0.01, betas=(0.9, 0.95), eps=1e-8, weight_decay=wd)
    for r in range(rounds):
        o.x[...] = o.xg[None] + RNG.standard_normal((K, P)) * 0.003        # local models after "H steps"
        q.grad = torch.tensor(o.xg - o.x.mean(axis=0))
        o.outer_sync()
        opt.step()
        np.testing.assert_allclose(o.xg, q.detach().numpy(), rtol=1e-10, atol=1e-14)
        for k in range(K):
            assert np.array_equal(o.x[k], o.xg)
    st = opt.state[q]
    np.testing.assert_allclose(o.u, st["exp_avg"].numpy(), rtol=1e-9, atol=1e-16)
    np.testing.assert_allclose(o.uv, st["exp_avg_sq"].numpy(), rtol=1e-9, atol=1e-20)
    assert o.n_outer == rounds


def test_adamw_outer_first_round_closed_form():
    # n = 1: m_hat = Delta, v_hat = Delta^2  =>  x_new = x (1 - lr wd) - lr * Delta / (|Delta| + eps)
    K, P, lr, wd, eps = 2, 40, 0.05, 0.1, 1e-8
    x0, o = _mk(K, P, outer_opt=1, outer_lr=lr, outer_weight_decay=wd, outer_eps=eps)
    xg = o.xg.copy()
    delta = xg - o.x.mean(axis=0)
    o.outer_sync()
    np.testing.assert_allclose(o.xg, xg * (1 - lr * wd) - lr * delta / (np.abs(delta) + eps), rtol=1e-12)


def test_sgd_outer_with_step_one_is_the_replica_mean():
    K, P = 4, 33
    x0, o = _mk(K, P, outer_opt=0, outer_lr=1.0, outer_momentum=0.0, outer_nesterov=False)
    mean = o.x.mean(axis=0)
    o.outer_sync()
    np.testing.assert_allclose(o.xg, mean, rtol=1e-13, atol=1e-16)


def test_outer_learning_rate_is_an_input_of_each_round():
    K, P = 2, 20
    x0, o = _mk(K, P, outer_lr=0.7, outer_momentum=0.9, outer_nesterov=True)
    q = torch.tensor(o.xg.astype(np.float64).copy(), requires_grad=True)
    opt = torch.optim.SGD([q], lr=0.7, momentum=0.9, nesterov=True)
    for r, lr in enumerate([0.1, 0.4, 0.7, 0.35, 0.0]):
        o.x[...] = o.xg[None] + RNG.standard_normal((K, P)) * 0.01
        q.grad = torch.tensor(o.xg - o.x.mean(axis=0))
        o.set_outer_lr(lr)
        for grp in opt.param_groups:
            grp["lr"] = lr
        o.outer_sync(); opt.step()
        np.testing.assert_allclose(o.xg, q.detach().numpy(), rtol=1e-11, atol=1e-15)


@pytest.mark.parametrize("warmup,total,sf,eta_min", [(10, 200, 0.1, 0.0), (5, 50, 1e-3, 0.02), (0, 30, 1.0, 0.0)])
def test_warm_up_then_cosine_matches_torch_schedulers(warmup, total, sf, eta_min):
    base = 0.8
    q = torch.zeros(1, requires_grad=True)
    opt = torch.optim.SGD([q], lr=base)
    cos = torch.optim.lr_scheduler.CosineAnnealingLR(opt, T_max=total - warmup, eta_min=eta_min)
    if warmup:
        lin = torch.optim.lr_scheduler.LinearLR(opt, start_factor=sf, end_factor=1.0, total_iters=warmup)
        sched = torch.optim.lr_scheduler.SequentialLR(opt, [lin, cos], milestones=[warmup])
    else:
        sched = cos
    for t in range(total + 1):
        want = opt.param_groups[0]["lr"]
        got = oracle.schedule(1, t, warmup, total, base, eta_min, sf)
        assert got == pytest.approx(want, rel=1e-9, abs=1e-12), t
        opt.step(); sched.step()
    assert oracle.schedule(1, total + 50, warmup, total, base, eta_min, sf) == pytest.approx(eta_min, abs=1e-15)


def test_schedule_closed_form_points():
    assert oracle.schedule(0, 0, 10, 100, 2.0, 0.0, 0.0) == 0.0
    assert oracle.schedule(0, 5, 10, 100, 2.0, 0.0, 0.0) == 1.0
    assert oracle.schedule(0, 10, 10, 100, 2.0) == 2.0 and oracle.schedule(0, 10**6, 10, 100, 2.0) == 2.0
    assert oracle.schedule(1, 55, 10, 100, 2.0, 0.0) == pytest.approx(1.0, abs=1e-15)      # half way down
    assert oracle.schedule(1, 100, 10, 100, 2.0, 0.5) == pytest.approx(0.5, abs=1e-15)
    assert oracle.schedule(1, 10, 10, 100, 2.0, 0.5) == 2.0
    assert math.isclose(oracle.schedule(1, 32, 10, 100, 1.0), (1 + math.cos(math.pi * 22 / 90)) / 2, rel_tol=1e-15)
