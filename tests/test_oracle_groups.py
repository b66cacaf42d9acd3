"""Pins for the two-level sum of the outer sync (workers spread over several machines: Algorithm 1's
All-Reduce across workers, an average by Sec. 2.2).  Grouping only changes the order in which the K
local models are added, so: one group, and K groups of one worker, are the plain ascending sum bit for
bit; inputs whose sums are exact in binary32 give the same bits for every grouping; in binary64 the
groupings agree to rounding; and every grouping stays within the rounding bound of the exact mean."""
from fractions import Fraction

import numpy as np
import pytest

import oracle


def _run(x0, groups, dtype="f32", rounds=2, **kw):
    K = x0.shape[0]
    o = oracle.Oracle(x0, K=K, H=1, p=0.0, dtype=dtype, **kw)
    o.set_sum_groups(groups)
    rng = np.random.default_rng(2)
    for _ in range(rounds):
        o.x[:] = o.x + (rng.standard_normal(o.x.shape) * 1e-3).astype(o.x.dtype)    # let the workers drift apart
        o.outer_sync()
    return o


@pytest.mark.parametrize("K", [2, 4, 6, 8])
def test_one_group_and_K_groups_are_the_plain_ascending_sum(K):
    x0 = (np.random.default_rng(1).standard_normal((K, 257)) * 0.02).astype(np.float32)
    ref = _run(x0, 0)
    for groups in (1, K):
        o = _run(x0, groups)
        for name in ("x", "xg", "u"):
            assert np.array_equal(getattr(o, name), getattr(ref, name)), (groups, name)


def test_exactly_summable_inputs_do_not_depend_on_the_grouping():
    # multiples of 2^-12 below 8: every partial sum of 8 of them is exact in binary32
    rng = np.random.default_rng(3)
    x0 = (rng.integers(-2**14, 2**14, size=(8, 300)) * 2.0 ** -12).astype(np.float32)
    outs = []
    for groups in (0, 2, 4, 8):
        o = oracle.Oracle(x0, K=8, H=1, p=0.0)
        o.set_sum_groups(groups)
        o.outer_sync()
        outs.append((o.xg.copy(), o.u.copy(), o.x.copy()))
    for xg, u, x in outs[1:]:
        assert np.array_equal(xg, outs[0][0]) and np.array_equal(u, outs[0][1]) and np.array_equal(x, outs[0][2])


def test_groupings_agree_to_rounding_and_respect_the_bound_of_the_exact_mean():
    K, P = 8, 64
    x0 = (np.random.default_rng(5).standard_normal((K, P)) * 0.02).astype(np.float32)
    for groups in (2, 4):
        o32 = oracle.Oracle(x0, K=K, H=1, p=0.0, outer_lr=1.0, outer_momentum=0.0, outer_nesterov=False)
        o32.set_sum_groups(groups)
        xg0 = o32.xg.copy()
        o32.outer_sync()                         # plain averaging: x_g <- x_g - (x_g - mean) ~ mean
        for i in range(P):
            exact = sum(Fraction(float(v)) for v in x0[:, i]) / K
            bound = (K + 2) * 2.0 ** -24 * float(sum(abs(Fraction(float(v))) for v in x0[:, i]) / K) + 2.0 ** -24 * abs(float(xg0[i]))
            assert abs(Fraction(float(o32.xg[i])) - exact) <= bound
        a = _run(x0, groups, dtype="f64")
        b = _run(x0, 0, dtype="f64")
        assert np.max(np.abs(a.xg - b.xg)) <= 1e-15


def test_two_groups_differ_from_one_level_somewhere_in_binary32():
    # the grouping is not a no-op: with generic data some elements round differently
    x0 = (np.random.default_rng(8).standard_normal((8, 4096)) * 0.02).astype(np.float32)
    a, b = _run(x0, 2, rounds=1), _run(x0, 0, rounds=1)
    assert not np.array_equal(a.xg, b.xg)
    assert np.max(np.abs(a.xg - b.xg)) < 1e-8


def test_uneven_groups_are_rejected():
    o = oracle.Oracle(np.zeros((6, 4), dtype=np.float32), K=6, H=1, p=0.0)
    with pytest.raises(ValueError):
        o.set_sum_groups(4)


def test_initial_global_model_uses_the_same_two_level_sum():
    rng = np.random.default_rng(11)
    x0 = (rng.standard_normal((6, 500)) * 0.02).astype(np.float32)
    plain = oracle.Oracle(x0, K=6, H=1, p=0.0)
    two = oracle.Oracle(x0, K=6, H=1, p=0.0, sum_groups=2)
    six = oracle.Oracle(x0, K=6, H=1, p=0.0, sum_groups=6)
    assert np.array_equal(six.xg, plain.xg)                          # K groups of one worker: the plain sum
    f = np.float32
    want = (((x0[0] + x0[1]) + x0[2]) + ((x0[3] + x0[4]) + x0[5])) / f(6)      # numpy's binary32 operations
    assert np.array_equal(two.xg, want)
    assert not np.array_equal(two.xg, plain.xg) and np.max(np.abs(two.xg - plain.xg)) < 1e-8
    exact = np.array([float(sum(Fraction(float(v)) for v in x0[:, i]) / 6) for i in range(500)])
    assert np.max(np.abs(two.xg.astype(np.float64) - exact)) <= 8 * 2.0 ** -24 * np.max(np.abs(x0))


@pytest.mark.parametrize("precision", [0, 1])
def test_ddp_step_sums_the_gradients_in_the_same_two_levels(precision):
    import workloads as W
    K, P = 6, 700
    rng = np.random.default_rng(21)
    x0 = np.tile((rng.standard_normal(P) * 0.02).astype(np.float32), (K, 1))
    g = (rng.standard_normal((K, P)) * 0.01).astype(np.float32)
    gin = W.bf16_bits_from_f32_host(g) if precision else g
    gval = (gin.astype(np.uint32) << 16).view(np.float32) if precision else g        # the values the step sees
    runs = {G: oracle.Oracle(x0, K=K, H=10**6, p=0.0, precision=precision, sum_groups=G) for G in (0, 1, 2, 3, 6)}
    for o in runs.values():
        o.ddp_step(gin, 1e-3)
    for G in (1, 6):                                   # one group / one worker per group: the plain sum
        for name in ("x", "m", "v", "xg"):
            assert np.array_equal(getattr(runs[G], name), getattr(runs[0], name)), (G, name)
    # first AdamW step from zero moments: m = (1 - beta1) * gbar, so m / (1 - beta1) recovers the averaged gradient
    f = np.float32
    for G in (2, 3):
        per = K // G
        parts = []
        for gi in range(G):
            part = gval[gi * per].copy()
            for k in range(gi * per + 1, (gi + 1) * per):
                part = part + gval[k]
            parts.append(part)
        tot = parts[0]
        for part in parts[1:]:
            tot = tot + part
        gbar = tot / f(K)
        assert np.array_equal(runs[G].m[0], f(1.0 - 0.9) * gbar)
        assert np.max(np.abs(runs[G].m[0] - runs[0].m[0])) < 1e-9
    exact = np.array([float(sum(Fraction(float(v)) for v in gval[:, i]) / K) for i in range(P)])
    assert np.max(np.abs(runs[2].m[0].astype(np.float64) / 0.1 - exact)) <= 1e-8
