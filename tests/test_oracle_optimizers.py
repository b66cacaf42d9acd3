"""Pins for the oracle's optimizer arithmetic.

The paper names InnerOPT = AdamW or momentum SGD and OuterOPT = SGD with
Nesterov momentum (Sec. 4.3) without printing them; the oracle writes out the
textbook forms.  They are pinned here against torch.optim on the CPU (library
routines), against closed forms, and the pull against the EMA identity the
paper states after Eq. (2).
"""
import numpy as np
import pytest
import torch

import oracle

RNG = np.random.default_rng(42)


def _mk(K, P, dtype, **kw):
    x0 = (RNG.standard_normal((K, P)) * 0.02).astype(np.float32)
    cfg = dict(K=K, H=10**9, p=0.0, inner=0, beta1=0.9, beta2=0.999, eps=1e-8,
               weight_decay=0.01, momentum=0.0, outer_lr=0.7, outer_momentum=0.9,
               outer_nesterov=True, seed=1, precision=0)
    cfg.update(kw)
    return x0, oracle.Oracle(x0, dtype=dtype, **cfg)


@pytest.mark.parametrize("p", [0.0, 0.1, 0.5])
def test_adamw_gradient_branch_matches_torch_adamw_f64(p):
    # Eq. (1): the gradient step is InnerOPT with step size alpha / (1 - p)
    K, P, alpha, steps = 2, 257, 1e-3, 25
    x0, o = _mk(K, P, "f64", p=p)
    params = [torch.tensor(x0[k].astype(np.float64), requires_grad=True) for k in range(K)]
    opts = [torch.optim.AdamW([q], lr=alpha / (1 - p), betas=(0.9, 0.999), eps=1e-8,
                              weight_decay=0.01) for q in params]
    for t in range(steps):
        g = (RNG.standard_normal((K, P)) * 0.01).astype(np.float32)
        o.inner_step(g, alpha, 16.0, forced=[0] * K)
        for k in range(K):
            params[k].grad = torch.tensor(g[k].astype(np.float64))
            opts[k].step()
    for k in range(K):
        np.testing.assert_allclose(o.x[k], params[k].detach().numpy(), rtol=1e-11, atol=1e-15)
        st = opts[k].state[params[k]]
        np.testing.assert_allclose(o.m[k], st["exp_avg"].numpy(), rtol=1e-11, atol=1e-18)
        np.testing.assert_allclose(o.v[k], st["exp_avg_sq"].numpy(), rtol=1e-11, atol=1e-22)
    assert list(o.s) == [steps] * K and o.t == steps


def test_adamw_f32_instantiation_matches_torch_f32_within_1e6():
    K, P, alpha, steps = 1, 1001, 1e-3, 50
    x0, o = _mk(K, P, "f32")
    q = torch.tensor(x0[0].copy(), requires_grad=True)
    opt = torch.optim.AdamW([q], lr=alpha, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01)
    for t in range(steps):
        g = (RNG.standard_normal((K, P)) * 0.01).astype(np.float32)
        o.inner_step(g, alpha, 16.0)
        q.grad = torch.tensor(g[0]); opt.step()
    ref = q.detach().numpy()
    err = np.abs(o.x[0] - ref) / np.maximum(np.abs(ref), 1e-7 / 1e-6)
    assert err.max() <= 1e-6


@pytest.mark.parametrize("p", [0.0, 0.2])
def test_momentum_sgd_gradient_branch_matches_torch_sgd_f64(p):
    K, P, alpha, steps = 2, 130, 0.1, 30
    x0, o = _mk(K, P, "f64", p=p, inner=1, momentum=0.9, weight_decay=1e-4)
    params = [torch.tensor(x0[k].astype(np.float64), requires_grad=True) for k in range(K)]
    opts = [torch.optim.SGD([q], lr=alpha / (1 - p), momentum=0.9, weight_decay=1e-4)
            for q in params]
    for t in range(steps):
        g = (RNG.standard_normal((K, P)) * 1e-3).astype(np.float32)
        o.inner_step(g, alpha, 0.5, forced=[0] * K)
        for k in range(K):
            params[k].grad = torch.tensor(g[k].astype(np.float64)); opts[k].step()
    for k in range(K):
        np.testing.assert_allclose(o.x[k], params[k].detach().numpy(), rtol=1e-12, atol=1e-16)
        np.testing.assert_allclose(o.m[k], opts[k].state[params[k]]["momentum_buffer"].numpy(),
                                   rtol=1e-12, atol=1e-18)


def test_adamw_first_step_closed_form():
    # m1 = (1-b1) g, v1 = (1-b2) g^2 => m^ = g, v^ = g^2:
    # x1 = x0 (1 - lr wd) - lr g / (|g| + eps)
    K, P, alpha, p = 1, 64, 1e-3, 0.25
    x0, o = _mk(K, P, "f64", p=p, weight_decay=0.01)
    g = (RNG.standard_normal((K, P)) * 0.01).astype(np.float32)
    o.inner_step(g, alpha, 16.0, forced=[0])
    lr = alpha / (1 - p)
    gd = g[0].astype(np.float64)
    want = x0[0].astype(np.float64) * (1 - lr * 0.01) - lr * gd / (np.abs(gd) + 1e-8)
    np.testing.assert_allclose(o.x[0], want, rtol=1e-12)


def test_sgdm_constant_gradient_closed_form():
    # wd = 0, constant g: buf_n = g (1 - mu^n) / (1 - mu); x_n = x_0 - lr sum_j buf_j
    K, P, alpha, mu, n = 1, 16, 0.05, 0.9, 12
    x0, o = _mk(K, P, "f64", inner=1, momentum=mu, weight_decay=0.0)
    g = (RNG.standard_normal((K, P)) * 1e-3).astype(np.float32)
    for _ in range(n):
        o.inner_step(g, alpha, 1.0)
    gd = g[0].astype(np.float64)
    buf = gd * (1 - mu ** n) / (1 - mu)
    total = gd * sum((1 - mu ** j) / (1 - mu) for j in range(1, n + 1))
    np.testing.assert_allclose(o.m[0], buf, rtol=1e-12)
    np.testing.assert_allclose(o.x[0], x0[0].astype(np.float64) - alpha * total, rtol=1e-12)


@pytest.mark.parametrize("beta", [0.064, 0.25, 1.0 / 32, 1.0, 1.7])
def test_pull_is_the_ema_of_eq2_and_contracts_geometrically(beta):
    # EMA form after Eq. (2): x_k <- (1 - beta) x_k + beta x, beta = alpha eta / p.
    # Against a fixed global copy, n pulls leave (1 - beta)^n of the gap.
    K, P, n = 3, 50, 9
    alpha, p = 1e-3, 0.1
    eta = beta * p / alpha
    x0 = (RNG.standard_normal((K, P)) * 0.02).astype(np.float32)
    x0[1] += 0.01; x0[2] -= 0.03
    o = oracle.Oracle(x0, dtype="f64", K=K, H=10**9, p=p, seed=3)
    xg = o.xg.copy()
    gap0 = o.x - xg
    m0, v0 = o.m.copy(), o.v.copy()
    for _ in range(n):
        o.inner_step(np.zeros((K, P), np.float32), alpha, eta, forced=[1] * K)
    np.testing.assert_allclose(o.x - xg, (1 - beta) ** n * gap0, rtol=1e-9, atol=1e-18)
    # a pull touches nothing but x_k
    assert np.array_equal(o.xg, xg) and np.array_equal(o.m, m0) and np.array_equal(o.v, v0)
    assert list(o.s) == [0] * K and o.t == n and list(o.last_b) == [1] * K


def test_pull_with_beta_one_lands_on_global_model_f32():
    K, P = 2, 300
    x0 = (RNG.standard_normal((K, P)) * 0.02).astype(np.float32)
    o = oracle.Oracle(x0, dtype="f32", K=K, H=10**9, p=0.5, seed=3)
    gap = np.abs(x0 - o.xg)
    o.pseudo_sync(0b11, 1.0)
    # x - 1*(x - xg): two roundings (of the gap, of the result) away from xg at most
    bound = 0.5 * np.spacing(gap.astype(np.float32)) + 0.5 * np.spacing(np.abs(o.xg))
    assert np.all(np.abs(o.x.astype(np.float64) - o.xg) <= bound.astype(np.float64) * 1.0000001)


def test_pseudo_sync_entry_uses_mask_and_changes_no_counter():
    K, P = 4, 33
    x0 = (RNG.standard_normal((K, P)) * 0.02).astype(np.float32)
    o = oracle.Oracle(x0, dtype="f64", K=K, H=10**9, p=0.1, seed=3)
    before = o.x.copy()
    o.pseudo_sync(0b0101, 0.25)
    for k in range(K):
        if k in (0, 2):
            np.testing.assert_allclose(o.x[k], 0.75 * before[k] + 0.25 * o.xg, rtol=1e-12)
        else:
            assert np.array_equal(o.x[k], before[k])
    assert o.t == 0 and list(o.s) == [0] * K and o.n_outer == 0


@pytest.mark.parametrize("nesterov", [True, False])
def test_outer_update_matches_torch_sgd_fed_with_delta(nesterov):
    # Eq. (3)/(4): Delta = x - average_k x_k is the "gradient" given to OuterOPT
    K, P, rounds, lr, mu = 4, 97, 6, 0.7, 0.9
    x0 = np.tile((RNG.standard_normal(P) * 0.02).astype(np.float32), (K, 1))
    o = oracle.Oracle(x0, dtype="f64", K=K, H=10**9, p=0.0, outer_lr=lr, outer_momentum=mu,
                      outer_nesterov=nesterov, seed=3)
    q = torch.tensor(o.xg.copy(), requires_grad=True)
    opt = torch.optim.SGD([q], lr=lr, momentum=mu, nesterov=nesterov)
    for r in range(rounds):
        o.x[...] = o.xg + RNG.standard_normal((K, P)) * 1e-3      # diverged local models
        m_before = o.m.copy()
        delta = o.xg - o.x.mean(axis=0)
        o.outer_sync()
        q.grad = torch.tensor(delta); opt.step()
        np.testing.assert_allclose(o.xg, q.detach().numpy(), rtol=1e-11, atol=1e-16)
        np.testing.assert_allclose(o.u, opt.state[q]["momentum_buffer"].numpy(), rtol=1e-10, atol=1e-18)
        for k in range(K):                                          # reset to the new global model
            assert np.array_equal(o.x[k], o.xg)
        assert np.array_equal(o.m, m_before)                        # inner state untouched
    assert o.n_outer == rounds


def test_outer_sgd_with_step_one_is_plain_averaging():
    # Theorem 1's setting: OuterOPT = SGD with step size 1 -> x <- average of local models
    K, P = 5, 40
    x0 = (RNG.standard_normal((K, P)) * 0.02).astype(np.float32)
    o = oracle.Oracle(x0, dtype="f64", K=K, H=10**9, p=0.0, outer_lr=1.0, outer_momentum=0.0,
                      outer_nesterov=False, seed=3)
    o.x[...] += RNG.standard_normal((K, P)) * 1e-2
    mean = o.x.mean(axis=0)
    o.outer_sync()
    np.testing.assert_allclose(o.xg, mean, rtol=1e-12, atol=1e-17)
