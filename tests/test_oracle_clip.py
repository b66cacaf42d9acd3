"""Pins for the oracle's global-norm gradient clipping.

Appendix B states that the GPT-Neo runs clip their gradients and says no more
(no threshold, no formula); the oracle takes the convention of the software the paper ran
(PyTorch's clip_grad_norm_: coefficient max_norm / (norm + 1e-6), capped at 1,
one norm over the worker's whole gradient).  Pinned here: the sum of squares
against Python's exact summation, the clipped step against the library routine
followed by the library optimizer, closed forms, and the cases in which the
clip must be a no-op.
"""
import math
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle

RNG = np.random.default_rng(11)


def _mk(K, P, dtype="f64", **kw):
    x0 = np.tile((RNG.standard_normal(P) * 0.02).astype(np.float32), (K, 1))
    cfg = dict(K=K, H=10**9, p=0.0, inner=0, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01,
               momentum=0.0, outer_lr=0.7, outer_momentum=0.9, outer_nesterov=True, seed=3, precision=0)
    cfg.update(kw)
    return x0, oracle.Oracle(x0, dtype=dtype, **cfg)


@pytest.mark.parametrize("n", [0, 1, 7, 1000, 100003])
def test_sum_of_squares_is_the_exact_sum_rounded_once(n):
    g = (RNG.standard_normal(n) * np.exp(RNG.uniform(-20, 20, n))).astype(np.float32)   # wide dynamic range
    exact = sum(Fraction(float(v)) ** 2 for v in g) if n <= 1000 else None
    want = math.fsum(float(v) * float(v) for v in g)        # squares of binary32 values are exact in binary64
    assert oracle.sumsq(g) == want
    if exact is not None and n:
        assert abs(Fraction(want) - exact) <= Fraction(math.ulp(want)) / 2
    bits = (g.view(np.uint32) >> 16).astype(np.uint16)
    wide = (bits.astype(np.uint32) << 16).view(np.float32)
    assert oracle.sumsq(bits) == math.fsum(float(v) * float(v) for v in wide)
    g64 = g.astype(np.float64) * (1 + 2.0 ** -30)           # squares no longer exact in binary64
    if n <= 1000:
        ex = sum(Fraction(float(v)) ** 2 for v in g64)
        got = oracle.sumsq(g64)
        assert abs(Fraction(got) - ex) <= Fraction(math.ulp(got)) / 2 if n else got == 0.0


def test_sum_of_squares_does_not_depend_on_the_thread_count():
    g = (RNG.standard_normal(50001) * 3).astype(np.float32)
    before = oracle.get_threads()
    vals = []
    for nt in (1, 2, 3, 8):
        oracle.set_threads(nt)
        vals.append(oracle.sumsq(g))
    oracle.set_threads(before)
    assert len(set(vals)) == 1


def test_clip_coefficient_closed_forms():
    assert oracle.clip_coef(0.0, 1.0) == 1.0                          # zero gradient: 1 / 1e-6 capped at 1
    assert oracle.clip_coef(4.0, 5.0) == 1.0                          # norm 2 below the threshold
    assert oracle.clip_coef(16.0, 1.0) == 1.0 / (4.0 + 1e-6)
    assert oracle.clip_coef(1.0, 1.0) == 1.0 / (1.0 + 1e-6)           # at the threshold the 1e-6 term shows


@pytest.mark.parametrize("inner", [0, 1])
def test_clipped_step_matches_library_clip_then_library_optimizer(inner):
    K, P, alpha, max_norm, steps = 3, 211, 1e-3, 0.05, 15
    kw = dict(inner=inner, momentum=0.9 if inner else 0.0, max_grad_norm=max_norm)
    x0, o = _mk(K, P, **kw)
    params = [torch.tensor(x0[k].astype(np.float64), requires_grad=True) for k in range(K)]
    if inner == 0:
        opts = [torch.optim.AdamW([q], lr=alpha, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01) for q in params]
    else:
        opts = [torch.optim.SGD([q], lr=alpha, momentum=0.9, weight_decay=0.01) for q in params]
    clipped_some = unclipped_some = False
    for t in range(steps):
        scale = 0.01 if t % 3 else 1e-4                                # some steps above, some below the threshold
        g = (RNG.standard_normal((K, P)) * scale).astype(np.float32)
        o.inner_step(g, alpha, 16.0)
        for k in range(K):
            params[k].grad = torch.tensor(g[k].astype(np.float64))
            total = torch.nn.utils.clip_grad_norm_([params[k]], max_norm)
            assert float(total) ** 2 == pytest.approx(o.sumsq[k], rel=1e-12)
            clipped_some |= o.clipc[k] < 1.0
            unclipped_some |= o.clipc[k] == 1.0
            opts[k].step()
    assert clipped_some and unclipped_some
    for k in range(K):
        np.testing.assert_allclose(o.x[k], params[k].detach().numpy(), rtol=1e-10, atol=1e-15)


def test_threshold_above_the_norm_changes_nothing_bitwise():
    K, P = 2, 300
    x0, a = _mk(K, P, dtype="f32", max_grad_norm=1e6)
    b = oracle.Oracle(x0, dtype="f32", K=K, H=10**9, p=0.0, seed=3)
    for _ in range(6):
        g = (RNG.standard_normal((K, P)) * 0.01).astype(np.float32)
        a.inner_step(g, 1e-3, 16.0); b.inner_step(g, 1e-3, 16.0)
    assert np.array_equal(a.x, b.x) and np.array_equal(a.v, b.v)
    assert list(a.clipc) == [1.0] * K


def test_clipped_gradient_has_the_threshold_norm_plain_sgd():
    # plain SGD, no decay: x_new = x - alpha * c * g, so (x - x_new)/alpha is the clipped gradient
    K, P, alpha, max_norm = 1, 5000, 0.5, 0.25
    x0, o = _mk(K, P, inner=1, weight_decay=0.0, max_grad_norm=max_norm)
    g = (RNG.standard_normal((K, P)) * 3).astype(np.float32)
    o.inner_step(g, alpha, 1.0)
    gc = (x0[0].astype(np.float64) - o.x[0]) / alpha
    assert np.linalg.norm(gc) == pytest.approx(max_norm, rel=1e-5)
    assert np.allclose(gc / np.linalg.norm(gc), g[0] / np.linalg.norm(g[0].astype(np.float64)), atol=1e-9)


def test_pulling_workers_neither_use_nor_report_a_norm():
    K, P = 4, 64
    x0, o = _mk(K, P, dtype="f32", p=0.5, max_grad_norm=0.01)
    g = (RNG.standard_normal((K, P))).astype(np.float32)
    o.inner_step(g, 1e-3, 16.0, forced=[1, 0, 1, 0])
    assert o.sumsq[0] == 0.0 and o.sumsq[2] == 0.0
    assert o.sumsq[1] == oracle.sumsq(g[1]) and o.clipc[1] < 1.0


def test_each_worker_is_clipped_by_its_own_norm():
    K, P = 2, 128
    x0, o = _mk(K, P, inner=1, weight_decay=0.0, max_grad_norm=1.0)
    g = np.stack([np.full(P, 1e-3, np.float32), np.full(P, 10.0, np.float32)])
    o.inner_step(g, 0.1, 1.0)
    assert o.clipc[0] == 1.0
    assert o.clipc[1] == pytest.approx(1.0 / (10.0 * math.sqrt(P) + 1e-6), rel=1e-15)


def test_ddp_phase_clips_the_averaged_gradient():
    K, P, alpha, max_norm = 4, 150, 1e-3, 0.02
    x0, o = _mk(K, P, max_grad_norm=max_norm)
    q = torch.tensor(x0[0].astype(np.float64), requires_grad=True)
    opt = torch.optim.AdamW([q], lr=alpha, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01)
    for _ in range(8):
        g = (RNG.standard_normal((K, P)) * 0.01).astype(np.float32)
        o.ddp_step(g, alpha)
        q.grad = torch.tensor(g.astype(np.float64).mean(axis=0))
        torch.nn.utils.clip_grad_norm_([q], max_norm)
        opt.step()
        assert len(set(o.clipc)) == 1 and o.clipc[0] < 1.0
    for k in range(K):
        np.testing.assert_allclose(o.x[k], q.detach().numpy(), rtol=1e-10, atol=1e-15)


def test_forced_sums_of_squares_replay_a_sample_of_a_larger_run():
    K, P = 3, 4000
    x0, full = _mk(K, P, dtype="f32", max_grad_norm=0.05)
    idx = np.arange(0, P, 17)
    part = oracle.Oracle(x0[:, idx], dtype="f32", K=K, H=10**9, p=0.0, seed=3, max_grad_norm=0.05)
    for _ in range(5):
        g = (RNG.standard_normal((K, P)) * 0.01).astype(np.float32)
        full.inner_step(g, 1e-3, 16.0)
        part.force_sumsq([oracle.sumsq(g[k]) for k in range(K)])
        part.inner_step(g[:, idx], 1e-3, 16.0)
    assert np.array_equal(part.x, full.x[:, idx]) and np.array_equal(part.m, full.m[:, idx])
