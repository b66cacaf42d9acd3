"""Pins for the oracle's DDP warm-up step.

The paper starts every run with a DDP phase (Sec. 3.3; Sec. 4.1): plain
mini-batch training in which the K workers' gradients are averaged and every
worker applies the same InnerOPT step.  The oracle takes that step once and
writes it to all workers.  It is pinned here to library optimizers fed an
independently computed mean gradient, to the gradient branch of Algorithm 1 at
p = 0 (which it must equal when all workers see the same gradient), to exact
rational arithmetic, and to a hand-computed value.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle

RNG = np.random.default_rng(7)


def _mk(K, P, dtype="f64", same=True, **kw):
    if same:
        x0 = np.tile((RNG.standard_normal(P) * 0.02).astype(np.float32), (K, 1))
    else:
        x0 = (RNG.standard_normal((K, P)) * 0.02).astype(np.float32)
    cfg = dict(K=K, H=10**9, p=0.1, inner=0, beta1=0.9, beta2=0.999, eps=1e-8,
               weight_decay=0.01, momentum=0.0, outer_lr=0.7, outer_momentum=0.9,
               outer_nesterov=True, seed=3, precision=0)
    cfg.update(kw)
    return x0, oracle.Oracle(x0, dtype=dtype, **cfg)


def test_hand_value_two_workers_plain_sgd():
    # x = 1, g = (1.0, 0.5): gbar = 0.75, alpha = 0.1 -> x = 1 - 0.075 = 0.925 for both workers and x_g
    x0 = np.ones((2, 1), dtype=np.float32)
    o = oracle.Oracle(x0, dtype="f64", K=2, H=4, p=0.5, inner=1, momentum=0.0, weight_decay=0.0, seed=1)
    o.ddp_step(np.array([[1.0], [0.5]], dtype=np.float32), 0.1)
    assert o.x[:, 0] == pytest.approx([0.925, 0.925], abs=1e-15)
    assert o.xg[0] == pytest.approx(0.925, abs=1e-15)
    assert o.t == 1 and list(o.s) == [1, 1] and list(o.last_b) == [0, 0] and o.n_outer == 0


@pytest.mark.parametrize("K", [1, 3, 8])
def test_adamw_ddp_equals_torch_adamw_on_the_mean_gradient(K):
    P, alpha, steps = 193, 1e-3, 20
    x0, o = _mk(K, P)
    q = torch.tensor(x0[0].astype(np.float64), requires_grad=True)
    opt = torch.optim.AdamW([q], lr=alpha, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01)
    for _ in range(steps):
        g = (RNG.standard_normal((K, P)) * 0.01).astype(np.float32)
        o.ddp_step(g, alpha)
        q.grad = torch.tensor(g.astype(np.float64).mean(axis=0))     # the mean, formed independently
        opt.step()
    ref = q.detach().numpy()
    st = opt.state[q]
    for k in range(K):
        np.testing.assert_allclose(o.x[k], ref, rtol=1e-11, atol=1e-15)
        np.testing.assert_allclose(o.m[k], st["exp_avg"].numpy(), rtol=1e-10, atol=1e-18)
        np.testing.assert_allclose(o.v[k], st["exp_avg_sq"].numpy(), rtol=1e-10, atol=1e-22)
    np.testing.assert_allclose(o.xg, ref, rtol=1e-11, atol=1e-15)
    assert list(o.s) == [steps] * K and o.t == steps


def test_momentum_sgd_ddp_equals_torch_sgd_on_the_mean_gradient():
    K, P, alpha, steps = 4, 77, 0.1, 25
    x0, o = _mk(K, P, inner=1, momentum=0.9, weight_decay=1e-4)
    q = torch.tensor(x0[0].astype(np.float64), requires_grad=True)
    opt = torch.optim.SGD([q], lr=alpha, momentum=0.9, weight_decay=1e-4)
    for _ in range(steps):
        g = (RNG.standard_normal((K, P)) * 1e-3).astype(np.float32)
        o.ddp_step(g, alpha)
        q.grad = torch.tensor(g.astype(np.float64).mean(axis=0)); opt.step()
    for k in range(K):
        np.testing.assert_allclose(o.x[k], q.detach().numpy(), rtol=1e-12, atol=1e-16)
        np.testing.assert_allclose(o.m[k], opt.state[q]["momentum_buffer"].numpy(), rtol=1e-11, atol=1e-18)


@pytest.mark.parametrize("inner", [0, 1])
@pytest.mark.parametrize("K", [1, 2, 4, 8])
def test_identical_gradients_reduce_to_the_gradient_branch_at_p_zero_bitwise(K, inner):
    # Gradients with 8 significant bits and K a power of two: every partial sum of K equal values and
    # the division by K are exact in binary32, so the averaged gradient IS the gradient, and the DDP
    # step must equal Algorithm 1's gradient step with step size alpha / (1 - 0) on every worker,
    # bit for bit.
    P, alpha = 301, 1e-3
    kw = dict(inner=inner, momentum=0.9 if inner else 0.0)
    x0, a = _mk(K, P, dtype="f32", **kw)
    b = oracle.Oracle(x0, dtype="f32", **{**dict(K=K, H=10**9, p=0.0, beta1=0.9, beta2=0.999, eps=1e-8,
                                                 weight_decay=0.01, seed=3), **kw})
    for _ in range(12):
        g1 = (RNG.standard_normal(P) * 0.01).astype(np.float32)
        g1 = (g1.view(np.uint32) & np.uint32(0xFFFF0000)).view(np.float32)
        g = np.tile(g1, (K, 1))
        a.ddp_step(g, alpha)
        b.inner_step(g, alpha, 16.0)
    assert np.array_equal(a.x, b.x) and np.array_equal(a.m, b.m)
    if inner == 0:
        assert np.array_equal(a.v, b.v)
    assert list(a.s) == list(b.s) and a.t == b.t


def test_exact_rational_arithmetic_momentum_sgd():
    K, P, alpha, mu, wd = 3, 2, 0.125, 0.5, 0.25
    x0 = np.tile(np.array([0.75, -1.5], dtype=np.float32), (K, 1))
    o = oracle.Oracle(x0, dtype="f64", K=K, H=10**9, p=0.3, inner=1, momentum=mu, weight_decay=wd, seed=1)
    F = Fraction
    x = [F(0.75), F(-1.5)]
    buf = [F(0), F(0)]
    for step in range(4):
        g = np.array([[(k + 1) * 0.25 * (-1) ** (i + step) for i in range(P)] for k in range(K)], dtype=np.float32)
        o.ddp_step(g, alpha)
        for i in range(P):
            gbar = sum(F(float(g[k, i])) for k in range(K)) / K
            gp = gbar + F(wd) * x[i]
            buf[i] = F(mu) * buf[i] + gp
            x[i] = x[i] - F(alpha) * buf[i]
    for k in range(K):
        for i in range(P):
            assert abs(o.x[k, i] - float(x[i])) <= 1e-14
            assert abs(o.m[k, i] - float(buf[i])) <= 1e-14


def test_state_is_taken_from_worker_zero_and_written_to_all():
    K, P = 3, 50
    x0, o = _mk(K, P, dtype="f32", same=False)          # slots differ: outside the DDP invariant
    g = (RNG.standard_normal((K, P)) * 0.01).astype(np.float32)
    u_before = o.u.copy()
    o.ddp_step(g, 1e-3)
    for k in range(1, K):
        assert np.array_equal(o.x[k], o.x[0]) and np.array_equal(o.m[k], o.m[0]) and np.array_equal(o.v[k], o.v[0])
    assert np.array_equal(o.xg, o.x[0]) and np.array_equal(o.u, u_before)
    # and it is worker 0's trajectory: a one-worker oracle started from slot 0 with the same mean gradient path
    one = oracle.Oracle(x0[:1], dtype="f32", K=1, H=10**9, p=0.1, seed=3)
    gbar = g[0].copy()
    for k in range(1, K):
        gbar = (gbar + g[k]).astype(np.float32)
    gbar = (gbar / np.float32(K)).astype(np.float32)
    one.ddp_step(gbar[None], 1e-3)
    assert np.array_equal(one.x[0], o.x[0])


def test_bf16_mode_follows_the_master_and_widens_gradients_exactly():
    K, P = 4, 400
    x0 = np.tile((RNG.standard_normal(P) * 0.02).astype(np.float32), (K, 1))
    common = dict(K=K, H=10**9, p=0.1, seed=5)
    a = oracle.Oracle(x0, dtype="f32", precision=1, **common)
    b = oracle.Oracle(x0, dtype="f32", precision=0, **common)
    for _ in range(5):
        g = (RNG.standard_normal((K, P)) * 0.01).astype(np.float32)
        bits = (g.view(np.uint32) >> 16).astype(np.uint16)
        wide = (bits.astype(np.uint32) << 16).view(np.float32)
        a.ddp_step(bits, 1e-3)
        b.ddp_step(wide, 1e-3)
    assert np.array_equal(a.x, b.x)
    for k in range(K):
        for i in range(0, P, 37):
            assert int(a.xw[k, i]) == oracle.bf16_from_f32(float(a.x[k, i]))


def test_warm_up_then_palsgd_phase_counts_steps_globally():
    # the decision stream is indexed by the global step t, which the warm-up steps advance
    K, P, W = 4, 10, 5
    x0, o = _mk(K, P, dtype="f32", p=0.5, H=4)
    for _ in range(W):
        o.ddp_step((RNG.standard_normal((K, P)) * 0.01).astype(np.float32), 1e-3)
    assert o.t == W and o.n_outer == 0
    o.step((RNG.standard_normal((K, P)) * 0.01).astype(np.float32), 1e-3, 16.0)
    assert list(o.last_b) == [oracle.decision(3, W, k, 0.5) for k in range(K)]
    for _ in range(2):
        o.step((RNG.standard_normal((K, P)) * 0.01).astype(np.float32), 1e-3, 16.0)
    assert o.t == 8 and o.n_outer == 1            # (t+1) mod H = 0 at global step index 7
