"""palsgd_outer_sync_noalloc against palsgd_outer_sync.

Some users of the library cannot allocate device memory at the point where they
synchronise (a framework's caching allocator owns the GPU's memory, or an
allocation's implicit device-wide synchronisation is not acceptable there), so
they cannot create a context.  The no-allocation entry point keeps its launch
tables in a fixed array inside the library instead.  This file checks that it
gives bit-identical results to the ordinary entry point, on two calls in a row
that use tensor lists of different shapes (the array keeps the first call's
tables when the second one starts), in both precisions, and that it refuses a
tensor list whose tables do not fit.

Collected last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest
import torch

import paper_2504_18454_b200 as P
import workloads as W
from workloads.configs import WorkloadConfig
from _harness import GpuRun, compare_state, make_oracle

pytestmark = pytest.mark.gpu


def _cfg(**kw):
    base = dict(name="noalloc", shape=lambda: [], K=4, H=10**6, p=0.25, eta=16.0, lr=1e-3, T=3)
    base.update(kw)
    return WorkloadConfig(**base)


def _diverged_run(cfg, numel, layout, seed):
    """A context whose K slots have drifted apart by a few inner steps."""
    Pn = int(sum(numel))
    rng = np.random.default_rng(seed)
    x0 = (rng.standard_normal((cfg.K, Pn)) * 0.02).astype(np.float32)
    run = GpuRun(cfg, x0, numel=numel, layout=layout)
    for t in range(cfg.T):
        g = np.stack([W.grads_host(Pn, cfg.grad_seed, t, k, cfg.grad_std) for k in range(cfg.K)])
        run.set_grads(W.bf16_bits_from_f32_host(g) if cfg.precision == 1 else g)
        run.inner_step(cfg.lr, cfg.eta)
    return run


def _copy_state(src: GpuRun, dst: GpuRun):
    names = ["param", "global_", "outer_mom"] + (["master"] if src.bf else [])
    for name in names:
        for row_s, row_d in zip(src.views[name], dst.views[name]):
            for a, b in zip(row_s, row_d):
                b.copy_(a)


def _noalloc_sync(run: GpuRun, cfg):
    v = run.views
    P.outer_sync_noalloc(K=cfg.K, numel=run.numel, params=v["param"], master=v.get("master"),
                         global_=v["global_"][0], outer_mom=v["outer_mom"][0], outer_lr=cfg.outer_lr,
                         outer_momentum=cfg.outer_momentum, outer_nesterov=cfg.outer_nesterov,
                         precision=cfg.precision, stream=run.stream)


def _assert_same(a: GpuRun, b: GpuRun):
    sa, sb = a.state(), b.state()
    for key in ("x", "xg", "u") + (("xw",) if a.bf else ()):
        assert np.array_equal(sa[key], sb[key]), key          # same kernel, same order: bit-identical
    assert a.guards_intact() and b.guards_intact()


@pytest.mark.parametrize("precision", [0, 1])
def test_two_calls_in_a_row_match_the_ordinary_outer_sync(precision):
    # first call: a ragged list over several blocks; second call: a shorter, differently shaped list,
    # a different K and the scalar (misaligned) path, so that stale tables would be noticed
    cases = [([8192 * 3 + 17, 5, 0, 4096, 1001], "separate", 4, 11),
             ([7, 12289], "misaligned", 3, 12)]
    for numel, layout, K, seed in cases:
        cfg = _cfg(K=K, precision=precision)
        ref = _diverged_run(cfg, numel, layout, seed)
        tst = _diverged_run(cfg, numel, layout, seed)
        _copy_state(ref, tst)
        for _ in range(2):                                     # two rounds: momentum carried over as well
            ref.outer_sync()
            _noalloc_sync(tst, cfg)
            _assert_same(ref, tst)
        st = tst.state()
        for k in range(K):
            assert np.array_equal(st["x"][k], st["xg"])        # every slot restarted from the global model


@pytest.mark.parametrize("precision", [0, 1])
def test_matches_the_cpu_oracle_directly(precision):
    # the same comparison every other parity test makes: CUDA against the oracle, element by element,
    # through two synchronisations with inner steps in between
    numel = [8192 * 2 + 9, 33, 0, 4100]
    Pn = int(sum(numel))
    cfg = _cfg(K=4, precision=precision)
    rng = np.random.default_rng(21)
    x0 = (rng.standard_normal((cfg.K, Pn)) * 0.02).astype(np.float32)
    run, orc = GpuRun(cfg, x0, numel=numel, layout="separate"), make_oracle(cfg, x0)
    for rnd in range(2):
        for t in range(cfg.T):
            g = np.stack([W.grads_host(Pn, cfg.grad_seed, rnd * cfg.T + t, k, cfg.grad_std) for k in range(cfg.K)])
            g = W.bf16_bits_from_f32_host(g) if precision == 1 else g
            run.set_grads(g); run.inner_step(cfg.lr, cfg.eta); orc.inner_step(g, cfg.lr, cfg.eta)
        _noalloc_sync(run, cfg)
        orc.outer_sync()
        compare_state(run.state(), orc, exact=True)
    assert run.guards_intact()


def test_refuses_a_capturing_stream():
    # under capture the table copy and the kernel node would be replayed with whatever later calls
    # left in the shared array, so the call must return ESTATE and enqueue nothing
    dev = torch.device("cuda:0")
    numel = [5000]
    cfg = _cfg(K=2)
    run = _diverged_run(cfg, numel, "arena", 3)
    before = run.state()
    side = torch.cuda.Stream(device=dev)
    v = run.views
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        graph.capture_begin()
        try:
            with pytest.raises(P.PalsgdError) as e:
                P.outer_sync_noalloc(K=cfg.K, numel=run.numel, params=v["param"], global_=v["global_"][0],
                                     outer_mom=v["outer_mom"][0], stream=side.cuda_stream)
        finally:
            graph.capture_end()
    assert e.value.status == -4
    torch.cuda.synchronize(dev)
    after = run.state()
    for key in before:
        assert np.array_equal(before[key], after[key]), key
    _noalloc_sync(run, cfg)                                    # and the entry point still works afterwards
    st = run.state()
    for k in range(cfg.K):
        assert np.array_equal(st["x"][k], st["xg"])


def test_plain_averaging_and_non_nesterov_momentum():
    numel = [9000, 33]
    for lr, mu, nesterov in ((1.0, 0.0, False), (0.5, 0.8, False)):
        cfg = _cfg(outer_lr=lr, outer_momentum=mu, outer_nesterov=nesterov)
        ref = _diverged_run(cfg, numel, "arena", 5)
        tst = _diverged_run(cfg, numel, "arena", 5)
        _copy_state(ref, tst)
        ref.outer_sync(); _noalloc_sync(tst, cfg)
        _assert_same(ref, tst)


def test_rejects_what_does_not_fit_and_bad_arguments():
    dev = torch.device("cuda:0")
    one = torch.zeros(8, device=dev)
    # 16 bytes of chunk table per 8192 elements: 2^20 bytes of scratch end below 2^29 + 2^25 elements.
    # Validation happens before any GPU work, so the (small) tensors are never touched.
    too_big = [8192 * 70000]
    with pytest.raises(P.PalsgdError) as e:
        P.outer_sync_noalloc(K=1, numel=too_big, params=[[one]], global_=[one], outer_mom=[one])
    assert e.value.status == -8
    with pytest.raises(P.PalsgdError) as e:
        P.outer_sync_noalloc(K=0, numel=[8], params=[], global_=[one], outer_mom=[one])
    assert e.value.status == -1
    with pytest.raises(P.PalsgdError) as e:                    # mixed precision needs the masters
        P.outer_sync_noalloc(K=1, numel=[8], params=[[one]], global_=[one], outer_mom=[one], precision=1)
    assert e.value.status == -1
    torch.cuda.synchronize(dev)
