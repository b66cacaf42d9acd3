"""Pins for the oracle's control flow: Algorithm 1 as a whole.

What the paper fixes: p -> 0 gives DiLoCo / Local SGD (Sec. 1, Sec. 6); every
worker restarts from the same global model at a sync (Sec. 3.1; the appendix's
"Xi_t = 0"); the mean dynamics of the appendix's "Basic Definitions"; the
branch coefficients alpha/(1-p) and alpha*eta/p of Eq. (1)/(2).  Plus a hand
trace and an exact-rational brute force on tiny inputs.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle

RNG = np.random.default_rng(123)


def _grads(K, P, std=0.01):
    return (RNG.standard_normal((K, P)) * std).astype(np.float32)


# ---------------------------------------------------------------- hand trace
def test_hand_trace_two_workers_one_parameter():
    """K=2, P=1, plain SGD inner (no momentum, no decay), alpha=0.1, p=0.5,
    eta=1 => pull coefficient beta = 0.1*1/0.5 = 0.2, gradient step size
    0.1/(1-0.5) = 0.2.  H=2, outer Nesterov lr 0.7, momentum 0.9.  x=(1,1), x_g=1.

    t=0: w0 pulls: 1 - 0.2(1-1) = 1.        w1 grad 0.5: 1 - 0.2*0.5 = 0.9
    t=1: w0 grad 1.0: 1 - 0.2 = 0.8.        w1 pulls: 0.9 - 0.2(0.9-1) = 0.92
    sync: mean 0.86, Delta = 1-0.86 = 0.14, u = 0.14,
          x_g = 1 - 0.7(0.14 + 0.9*0.14) = 1 - 0.7*0.266 = 0.8138; slots = 0.8138
    t=2: both grad 0.5: 0.8138 - 0.1 = 0.7138
    t=3: w0 pulls: 0.7138 - 0.2(0.7138-0.8138) = 0.7338;  w1 grad 0.1: 0.6938
    sync: mean 0.7138, Delta = 0.1, u = 0.9*0.14 + 0.1 = 0.226,
          x_g = 0.8138 - 0.7(0.1 + 0.9*0.226) = 0.8138 - 0.7*0.3034 = 0.60142
    """
    x0 = np.ones((2, 1), np.float32)
    o = oracle.Oracle(x0, dtype="f64", K=2, H=2, p=0.5, inner=1, momentum=0.0, weight_decay=0.0,
                      outer_lr=0.7, outer_momentum=0.9, outer_nesterov=True)
    g = lambda a, b: np.array([[a], [b]], np.float32)
    o.step(g(0.0, 0.5), 0.1, 1.0, forced=[1, 0])
    np.testing.assert_allclose(o.x.ravel(), [1.0, 0.9], rtol=1e-7)
    assert o.n_outer == 0 and list(o.s) == [0, 1]
    o.step(g(1.0, 0.0), 0.1, 1.0, forced=[0, 1])
    np.testing.assert_allclose(o.x.ravel(), [0.8138, 0.8138], rtol=1e-7)
    np.testing.assert_allclose(o.xg, [0.8138], rtol=1e-7)
    np.testing.assert_allclose(o.u, [0.14], rtol=1e-7)
    assert o.n_outer == 1 and list(o.s) == [1, 1] and o.t == 2
    o.step(g(0.5, 0.5), 0.1, 1.0, forced=[0, 0])
    np.testing.assert_allclose(o.x.ravel(), [0.7138, 0.7138], rtol=1e-7)
    o.step(g(0.0, 0.1), 0.1, 1.0, forced=[1, 0])
    np.testing.assert_allclose(o.u, [0.226], rtol=1e-7)
    np.testing.assert_allclose(o.xg, [0.60142], rtol=1e-7)
    np.testing.assert_allclose(o.x.ravel(), [0.60142, 0.60142], rtol=1e-7)
    assert o.n_outer == 2 and list(o.s) == [2, 3] and o.t == 4


# ------------------------------------------------------- exact brute force
def _rational_palsgd(x0, grads, decisions, *, H, p, alpha, eta, mu_in, wd, lr_out, mu_out, nesterov):
    """Algorithm 1 in exact rationals (momentum-SGD inner, Nesterov outer)."""
    K, P = len(x0), len(x0[0])
    F = Fraction
    x = [[F(v) for v in row] for row in x0]
    buf = [[F(0)] * P for _ in range(K)]
    xg = [sum(x[k][i] for k in range(K)) / K for i in range(P)]
    u = [F(0)] * P
    for t, (g, b) in enumerate(zip(grads, decisions)):
        for k in range(K):
            for i in range(P):
                if b[k]:
                    x[k][i] = x[k][i] - alpha * eta / p * (x[k][i] - xg[i])
                else:
                    gp = F(g[k][i]) + wd * x[k][i]
                    buf[k][i] = mu_in * buf[k][i] + gp
                    x[k][i] = x[k][i] - alpha / (1 - p) * buf[k][i]
        if (t + 1) % H == 0:
            for i in range(P):
                delta = xg[i] - sum(x[k][i] for k in range(K)) / K
                u[i] = mu_out * u[i] + delta
                xg[i] = xg[i] - lr_out * ((delta + mu_out * u[i]) if nesterov else u[i])
                for k in range(K):
                    x[k][i] = xg[i]
    return x, buf, xg, u


@pytest.mark.parametrize("nesterov", [True, False])
def test_tiny_run_matches_exact_rational_arithmetic(nesterov):
    K, P, H, T = 3, 4, 3, 8          # T not a multiple of H: two syncs, two trailing steps
    F = Fraction
    hp = dict(H=H, p=F(1, 4), alpha=F(1, 8), eta=F(1, 2), mu_in=F(1, 2), wd=F(1, 16),
              lr_out=F(3, 4), mu_out=F(1, 2), nesterov=nesterov)
    x0 = RNG.integers(-64, 64, size=(K, P)) / 64.0
    grads = RNG.integers(-32, 32, size=(T, K, P)) / 128.0
    dec = RNG.integers(0, 2, size=(T, K))
    dec[0] = [1, 0, 1]; dec[1] = [0, 0, 0]
    want = _rational_palsgd(x0.tolist(), grads.tolist(), dec.tolist(), **hp)
    o = oracle.Oracle(x0.astype(np.float32), dtype="f64", K=K, H=H, p=0.25, inner=1, momentum=0.5,
                      weight_decay=1 / 16, outer_lr=0.75, outer_momentum=0.5,
                      outer_nesterov=nesterov)
    for t in range(T):
        o.step(grads[t].astype(np.float32), 1 / 8, 1 / 2, forced=dec[t])
    tof = lambda a: np.array([[float(v) for v in r] for r in a]) if isinstance(a[0], list) \
        else np.array([float(v) for v in a])
    np.testing.assert_allclose(o.x, tof(want[0]), rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(o.m, tof(want[1]), rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(o.xg, tof(want[2]), rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(o.u, tof(want[3]), rtol=1e-12, atol=1e-15)
    assert o.n_outer == T // H and o.t == T
    assert list(o.s) == list((1 - dec).sum(axis=0))


# ----------------------------------------------------- reductions the paper fixes
def test_p_zero_is_diloco_k_independent_adamw_runs_plus_outer_nesterov():
    K, P, H, T, alpha = 3, 120, 4, 12, 1e-3
    x_init = (RNG.standard_normal(P) * 0.02).astype(np.float32)
    o = oracle.Oracle(np.tile(x_init, (K, 1)), dtype="f64", K=K, H=H, p=0.0, seed=77,
                      outer_lr=0.7, outer_momentum=0.9)
    # reference built from library optimizers only
    xg = torch.tensor(x_init.astype(np.float64), requires_grad=True)
    outer = torch.optim.SGD([xg], lr=0.7, momentum=0.9, nesterov=True)
    loc = [xg.detach().clone().requires_grad_(True) for _ in range(K)]
    inner = [torch.optim.AdamW([q], lr=alpha, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01)
             for q in loc]
    for t in range(T):
        g = _grads(K, P)
        o.step(g, alpha, 16.0)
        assert list(o.last_b) == [0] * K           # p = 0: no pull, ever
        for k in range(K):
            loc[k].grad = torch.tensor(g[k].astype(np.float64)); inner[k].step()
        if (t + 1) % H == 0:
            xg.grad = xg.detach() - torch.stack([q.detach() for q in loc]).mean(0)
            outer.step()
            with torch.no_grad():
                for q in loc:
                    q.copy_(xg)                      # inner optimizer state is kept
    np.testing.assert_allclose(o.xg, xg.detach().numpy(), rtol=1e-10, atol=1e-15)
    for k in range(K):
        np.testing.assert_allclose(o.x[k], loc[k].detach().numpy(), rtol=1e-10, atol=1e-15)
    assert o.n_outer == T // H


def test_p_zero_outer_sgd_step_one_is_local_sgd_averaging():
    K, P, H, alpha = 4, 64, 5, 0.05
    x_init = (RNG.standard_normal(P) * 0.02).astype(np.float32)
    o = oracle.Oracle(np.tile(x_init, (K, 1)), dtype="f64", K=K, H=H, p=0.0, inner=1, momentum=0.0,
                      weight_decay=0.0, outer_lr=1.0, outer_momentum=0.0, outer_nesterov=False)
    x = np.tile(x_init.astype(np.float64), (K, 1))
    for t in range(2 * H):
        g = _grads(K, P)
        o.step(g, alpha, 1.0)
        x -= alpha * g.astype(np.float64)
        if (t + 1) % H == 0:
            x[...] = x.mean(axis=0)
    np.testing.assert_allclose(o.x, x, rtol=1e-11, atol=1e-16)
    np.testing.assert_allclose(o.xg, x[0], rtol=1e-11, atol=1e-16)


@pytest.mark.parametrize("inner", [0, 1])
def test_single_worker_h1_plain_averaging_is_the_plain_inner_optimizer(inner):
    P, T, alpha = 200, 20, 1e-2
    x_init = (RNG.standard_normal(P) * 0.02).astype(np.float32)
    o = oracle.Oracle(x_init[None], dtype="f64", K=1, H=1, p=0.0, inner=inner, momentum=0.9,
                      weight_decay=0.01, outer_lr=1.0, outer_momentum=0.0, outer_nesterov=False)
    q = torch.tensor(x_init.astype(np.float64), requires_grad=True)
    opt = (torch.optim.AdamW([q], lr=alpha, weight_decay=0.01) if inner == 0 else
           torch.optim.SGD([q], lr=alpha, momentum=0.9, weight_decay=0.01))
    for t in range(T):
        g = _grads(1, P)
        o.step(g, alpha, 16.0)
        q.grad = torch.tensor(g[0].astype(np.float64)); opt.step()
    np.testing.assert_allclose(o.x[0], q.detach().numpy(), rtol=1e-10, atol=1e-15)
    np.testing.assert_allclose(o.xg, q.detach().numpy(), rtol=1e-10, atol=1e-15)
    assert o.n_outer == T


# ------------------------------------------------------------ invariants
@pytest.mark.parametrize("dtype", ["f32", "f64"])
def test_consensus_and_mean_after_sync(dtype):
    K, P, H = 5, 301, 6
    x0 = (RNG.standard_normal((K, P)) * 0.02).astype(np.float32)      # slots differ at start
    o = oracle.Oracle(x0, dtype=dtype, K=K, H=H, p=0.3, seed=9)
    # init: global copy is the fixed-order mean of the slots
    acc = x0[0].astype(o.x.dtype)
    for k in range(1, K):
        acc = acc + x0[k].astype(o.x.dtype)
    assert np.array_equal(o.xg, acc / o.x.dtype.type(K))
    for t in range(3 * H):
        o.step(_grads(K, P), 1e-3, 16.0)
        if (t + 1) % H == 0:
            for k in range(K):                                        # bitwise consensus
                assert np.array_equal(o.x[k], o.xg)
        elif (t + 1) % H == 1:
            assert not np.array_equal(o.x[0], o.x[1])                 # workers diverge again
    assert o.n_outer == 3


def test_plain_averaging_preserves_the_mean():
    K, P = 6, 128
    x0 = (RNG.standard_normal((K, P)) * 0.02).astype(np.float32)
    o = oracle.Oracle(x0, dtype="f64", K=K, H=10**9, p=0.0, outer_lr=1.0, outer_momentum=0.0,
                      outer_nesterov=False)
    o.x[...] += RNG.standard_normal((K, P)) * 0.01
    before = o.x.mean(axis=0)
    o.outer_sync()
    np.testing.assert_allclose(o.x.mean(axis=0), before, rtol=1e-12, atol=1e-17)


def test_mean_dynamics_between_syncs():
    """Appendix, "Basic Definitions" (SGD inner): with the per-worker effective
    gradient  (1-b_k)/(1-p) * g_k + (eta b_k / p)(x_k - x),
    the worker mean obeys  xbar(t+1) = xbar(t) - alpha * mean_k(effective gradient)."""
    K, P, H, alpha, eta, p, seed = 8, 64, 50, 0.05, 2.0, 0.3, 2025
    x0 = (RNG.standard_normal((K, P)) * 0.02).astype(np.float32)
    o = oracle.Oracle(x0, dtype="f64", K=K, H=H, p=p, inner=1, momentum=0.0, weight_decay=0.0,
                      seed=seed)
    seen = set()
    for t in range(H - 1):
        g = _grads(K, P)
        b = np.array([oracle.decision(seed, t, k, p) for k in range(K)], dtype=np.float64)
        seen.update(b.tolist())
        xk, xg = o.x.copy(), o.xg.copy()
        eff = ((1 - b) / (1 - p))[:, None] * g + (eta * b / p)[:, None] * (xk - xg)
        o.step(g, alpha, eta)
        assert np.array_equal(o.last_b, b.astype(np.uint8))
        np.testing.assert_allclose(o.x.mean(axis=0), xk.mean(axis=0) - alpha * eff.mean(axis=0),
                                   rtol=1e-11, atol=1e-16)
        assert np.array_equal(o.xg, xg)              # x^(t+1) = x^(t) between syncs
    assert seen == {0.0, 1.0}


def test_theory_coupling_alpha_eta_equals_p_over_2h():
    # Lemma 3's step-size coupling alpha*eta = p/(2H) makes the pull coefficient 1/(2H)
    K, P, H, p, alpha = 2, 16, 8, 0.25, 1e-2
    eta = p / (2 * H) / alpha
    x0 = (RNG.standard_normal((K, P)) * 0.02).astype(np.float32)
    o = oracle.Oracle(x0, dtype="f64", K=K, H=10**9, p=p)
    before = o.x.copy()
    o.inner_step(np.zeros((K, P), np.float32), alpha, eta, forced=[1, 1])
    np.testing.assert_allclose(o.x, before - (before - o.xg) / (2 * H), rtol=1e-12)


# ------------------------------------------------------- counters and branches
def test_step_counts_follow_gradient_steps_only_and_bias_correction_uses_them():
    # a worker that pulled first takes its FIRST AdamW step later: closed form of step one
    K, P, alpha, p = 2, 32, 1e-3, 0.5
    x0 = np.tile((RNG.standard_normal(P) * 0.02).astype(np.float32), (K, 1))
    o = oracle.Oracle(x0, dtype="f64", K=K, H=10**9, p=p, weight_decay=0.0)
    g0, g1 = _grads(K, P), _grads(K, P)
    o.inner_step(g0, alpha, 1.0, forced=[1, 0])
    assert list(o.s) == [0, 1] and list(o.last_b) == [1, 0]
    x_before = o.x[0].copy()
    o.inner_step(g1, alpha, 1.0, forced=[0, 0])
    assert list(o.s) == [1, 2] and o.t == 2
    gd = g1[0].astype(np.float64)
    np.testing.assert_allclose(o.x[0], x_before - alpha / (1 - p) * gd / (np.abs(gd) + 1e-8), rtol=1e-12)
    np.testing.assert_allclose(o.pow1, [0.9, 0.81], rtol=1e-15)


def test_branches_are_exclusive_and_gradient_is_ignored_on_pull():
    K, P = 1, 16
    x0 = (RNG.standard_normal((K, P)) * 0.02).astype(np.float32)
    a = oracle.Oracle(x0, dtype="f64", K=K, H=10**9, p=0.5)
    b = oracle.Oracle(x0, dtype="f64", K=K, H=10**9, p=0.5)
    a.x += 0.01; b.x += 0.01
    a.inner_step(_grads(K, P, 1.0), 1e-3, 16.0, forced=[1])
    b.inner_step(np.zeros((K, P), np.float32), 1e-3, 16.0, forced=[1])
    assert np.array_equal(a.x, b.x) and not a.m.any() and not a.v.any()


def test_undefined_coefficients_are_refused():
    x0 = np.zeros((1, 4), np.float32)
    o = oracle.Oracle(x0, K=1, H=4, p=0.0)
    with pytest.raises(ValueError):
        o.inner_step(np.zeros((1, 4), np.float32), 1e-3, 1.0, forced=[1])     # pull needs p > 0
    o = oracle.Oracle(x0, K=1, H=4, p=1.0)
    with pytest.raises(ValueError):
        o.inner_step(np.zeros((1, 4), np.float32), 1e-3, 1.0, forced=[0])     # gradient needs p < 1
    o.inner_step(np.zeros((1, 4), np.float32), 1e-3, 1.0)                     # p = 1 always pulls
    assert list(o.last_b) == [1]


# ------------------------------------------------------------ mixed precision
def test_bf16_mode_master_math_equals_fp32_mode_and_working_copy_is_rounded_master():
    from workloads import bf16_bits_from_f32_host
    K, P, H = 3, 500, 4
    x0 = (RNG.standard_normal((K, P)) * 0.02).astype(np.float32)
    a = oracle.Oracle(x0, dtype="f32", K=K, H=H, p=0.3, seed=4, precision=1)
    b = oracle.Oracle(x0, dtype="f32", K=K, H=H, p=0.3, seed=4, precision=0)
    rounded = lambda x: torch.from_numpy(x.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(a.xw, rounded(a.x))
    for t in range(2 * H + 1):
        g16 = bf16_bits_from_f32_host(_grads(K, P))
        g32 = (g16.astype(np.uint32) << 16).view(np.float32)              # exact widening
        a.step(g16, 1e-3, 16.0)
        b.step(g32, 1e-3, 16.0)
        assert np.array_equal(a.x, b.x) and np.array_equal(a.m, b.m) and np.array_equal(a.v, b.v)
        assert np.array_equal(a.xw, rounded(a.x))                          # after every master write
    assert np.array_equal(a.xg, b.xg) and np.array_equal(a.u, b.u)


def test_f32_instantiation_stays_close_to_f64():
    K, P, H, T = 4, 4096, 8, 32
    x0 = np.tile((RNG.standard_normal(P) * 0.02).astype(np.float32), (K, 1))
    a = oracle.Oracle(x0, dtype="f32", K=K, H=H, p=0.25, seed=2025)
    b = oracle.Oracle(x0, dtype="f64", K=K, H=H, p=0.25, seed=2025)
    for t in range(T):
        g = _grads(K, P)
        a.step(g, 1e-3, 16.0); b.step(g, 1e-3, 16.0)
    err = np.abs(a.x - b.x) / np.maximum(np.abs(b.x), 1e-7 / 1e-6)
    assert err.max() < 5e-6            # rounding only: a dropped term would be >= 1e-3
    assert np.array_equal(a.last_b, b.last_b) and list(a.s) == list(b.s)
