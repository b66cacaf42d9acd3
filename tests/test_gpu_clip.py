"""GPU parity of global-norm gradient clipping against the CPU oracle: the sums
of squares and clip coefficients bit for bit, and the clipped steps element by
element, in the Algorithm 1 phase and in the DDP warm-up phase."""
import numpy as np
import pytest
import torch

import oracle
import workloads as W
from workloads.configs import WorkloadConfig
from _harness import GpuRun, compare_state, make_oracle

pytestmark = pytest.mark.gpu

RAGGED = [1, 3, 7, 1001, 4095, 4096, 4097, 0, 5, 12289, 8]


def _cfg(**kw):
    base = dict(name="clip", shape=lambda: [], K=4, H=4, p=0.25, eta=16.0, lr=1e-3, T=10)
    base.update(kw)
    return WorkloadConfig(**base)


def _x0(K, P, seed=1):
    rng = np.random.default_rng(seed)
    return np.tile((rng.standard_normal(P) * 0.02).astype(np.float32), (K, 1))


def _grads(cfg, P, t, scale=1.0):
    g = np.stack([W.grads_host(P, cfg.grad_seed, t, k, cfg.grad_std) for k in range(cfg.K)]) * np.float32(scale)
    return W.bf16_bits_from_f32_host(g) if cfg.precision == 1 else g


def _check_norms(gpu, orc, which):
    ss, cl = gpu.grad_norms()
    for k in which:
        assert ss[k] == orc.sumsq[k], (k, ss[k], orc.sumsq[k])                 # exact sum, rounded once
        assert np.float32(cl[k]) == np.float32(orc.clipc[k]), (k, cl[k], orc.clipc[k])


def _run(cfg, numel, layout, max_norm, n_ddp=0, T=None, scales=(1.0, 0.05)):
    P = int(sum(numel))
    x0 = _x0(cfg.K, P)
    gpu, orc = GpuRun(cfg, x0, numel=numel, layout=layout), make_oracle(cfg, x0)
    gpu.set_grad_clip(max_norm); orc.set_grad_clip(max_norm)
    clipped = unclipped = 0
    for t in range(T if T is not None else cfg.T):
        g = _grads(cfg, P, t, scales[t % len(scales)])
        gpu.set_grads(g)
        if t < n_ddp:
            gpu.ddp_step(cfg.lr); orc.ddp_step(g, cfg.lr)
            took = range(cfg.K)
        else:
            gpu.step(cfg.lr, cfg.eta); orc.step(g, cfg.lr, cfg.eta)
            took = [k for k in range(cfg.K) if not orc.last_b[k]]
        _check_norms(gpu, orc, took)
        clipped += sum(orc.clipc[k] < 1.0 for k in took)
        unclipped += sum(orc.clipc[k] == 1.0 for k in took)
        c = gpu.counters()
        assert c["s"] == [int(v) for v in orc.s] and c["last_b"] == [int(v) for v in orc.last_b]
    compare_state(gpu.state(), orc, exact=True)
    assert gpu.guards_intact()
    return gpu, orc, clipped, unclipped


@pytest.mark.parametrize("layout", ["arena", "separate", "misaligned"])
@pytest.mark.parametrize("inner,precision", [(0, 0), (1, 0), (0, 1), (1, 1)])
def test_ragged_list_clipped_steps_match_oracle(layout, inner, precision):
    cfg = _cfg(inner=inner, precision=precision, momentum=0.9 if inner else 0.0)
    P = sum(RAGGED)
    thr = 0.3 * 0.01 * np.sqrt(P)                     # between the norms of the two gradient scales
    _, _, clipped, unclipped = _run(cfg, RAGGED, layout, thr)
    assert clipped > 0 and unclipped > 0


@pytest.mark.parametrize("inner,precision", [(0, 0), (1, 1)])
def test_ddp_phase_clips_the_averaged_gradient_then_local_phase(inner, precision):
    cfg = _cfg(inner=inner, precision=precision, momentum=0.9 if inner else 0.0, K=5)
    P = sum(RAGGED)
    thr = 0.3 * 0.01 * np.sqrt(P / 5)
    _, _, clipped, unclipped = _run(cfg, RAGGED, "arena", thr, n_ddp=5, T=11)
    assert clipped > 0 and unclipped > 0


@pytest.mark.parametrize("K", [1, 3, 8, 64])
def test_worker_counts(K):
    numel = [4096 * 2 + 13, 77]
    _run(_cfg(K=K, H=3), numel, "arena", 0.2, T=5)
    _run(_cfg(K=K, H=3, precision=1), numel, "arena", 0.2, n_ddp=2, T=4)


def test_sum_of_squares_is_exact_over_a_wide_dynamic_range():
    # gradients spanning 2^-60 .. 2^60: a plain binary64 accumulation in any order loses the small terms
    numel = [30000, 5]
    P = sum(numel)
    cfg = _cfg(K=3, p=0.0, H=10**6)
    rng = np.random.default_rng(5)
    gpu, orc = GpuRun(cfg, _x0(3, P), numel=numel), make_oracle(cfg, _x0(3, P))
    gpu.set_grad_clip(1.0); orc.set_grad_clip(1.0)
    for t in range(3):
        g = (rng.standard_normal((3, P)) * np.exp2(rng.integers(-60, 60, (3, P)))).astype(np.float32)
        gpu.set_grads(g); gpu.inner_step(1e-3, 16.0); orc.inner_step(g, 1e-3, 16.0)
        _check_norms(gpu, orc, range(3))
    compare_state(gpu.state(), orc, exact=True)


def _bf16_bits(a):
    return W.bf16_bits_from_f32_host(np.asarray(a, dtype=np.float32))


@pytest.mark.parametrize("kind", ["gaussian", "mostly_zero", "two_scales", "wide", "tiny_and_denormal", "one_outlier_late",
                                  "infinite"])
def test_bf16_sum_of_squares_is_exact_on_every_route(kind):
    # bf16 gradients take plain binary64 chains whose exactness is tested after the run (ordinary data), send
    # far-off elements through the double-double accumulator one by one, and redo an item in double-double when
    # the test fails (data spread over many binades): all three routes must give the exactly rounded sum
    numel = [8192 * 9 + 24, 40, 8192]
    P = sum(numel)
    cfg = _cfg(K=3, p=0.0, H=10**6, precision=1)
    rng = np.random.default_rng(17)
    gpu, orc = GpuRun(cfg, _x0(3, P), numel=numel), make_oracle(cfg, _x0(3, P))
    gpu.set_grad_clip(1.0); orc.set_grad_clip(1.0)
    for t in range(2):
        z = rng.standard_normal((3, P))
        if kind == "gaussian":
            g = z * 0.01
        elif kind == "mostly_zero":
            g = np.where(rng.random((3, P)) < 0.97, 0.0, z * 0.01)
        elif kind == "two_scales":                       # a few elements 2^-20 below the rest
            g = np.where(rng.random((3, P)) < 0.001, z * 0.01 * 2.0 ** -20, z * 0.01)
        elif kind == "wide":
            g = z * np.exp2(rng.integers(-60, 60, (3, P)))
        elif kind == "tiny_and_denormal":                # bf16 denormals (below 2^-126) among tiny normal values
            g = z * np.exp2(rng.integers(-133, -120, (3, P)))
        elif kind == "one_outlier_late":                 # the largest element arrives after the range was fixed
            g = z * 0.01
            g[:, P - 5] = 3.0e4
        else:
            g = z * 0.01
            g[1, 12345] = np.inf
        bits = _bf16_bits(g)
        gpu.set_grads(bits); gpu.inner_step(1e-3, 16.0); orc.inner_step(bits, 1e-3, 16.0)
        _check_norms(gpu, orc, range(3))
    if kind != "infinite":
        compare_state(gpu.state(), orc, exact=True)


def test_threshold_above_every_norm_is_bitwise_the_unclipped_run_and_costs_one_more_launch():
    numel = RAGGED
    P = sum(numel)
    cfg = _cfg(K=4, p=0.0)
    a, b = GpuRun(cfg, _x0(4, P), numel=numel), GpuRun(cfg, _x0(4, P), numel=numel)
    a.set_grad_clip(1e9)
    for t in range(4):
        g = _grads(cfg, P, t)
        a.set_grads(g); a.inner_step(cfg.lr, cfg.eta)
        b.set_grads(g); b.inner_step(cfg.lr, cfg.eta)
    sa, sb = a.state(), b.state()
    for key in sa:
        assert np.array_equal(sa[key], sb[key]), key
    assert a.lib.get_launch_count() == 1 + 2 * 4 and b.lib.get_launch_count() == 1 + 4
    a.set_grad_clip(0.0)                               # off again: one launch per step
    a.set_grads(_grads(cfg, P, 4)); a.inner_step(cfg.lr, cfg.eta)
    assert a.lib.get_launch_count() == 1 + 2 * 4 + 1


def test_launch_shape_independence():
    numel = RAGGED
    P = sum(numel)
    cfg = _cfg(K=8, H=3)
    outs, norms = [], []
    for caps in (None, (7, 3), (148 * 4, 148)):
        r = GpuRun(cfg, _x0(8, P), numel=numel)
        r.set_grad_clip(0.05)
        if caps:
            r.lib.set_tuning(0, caps[0]); r.lib.set_tuning(1, caps[1])
        for t in range(2):
            r.set_grads(_grads(cfg, P, t)); r.ddp_step(cfg.lr)
        for t in range(2, 6):
            r.set_grads(_grads(cfg, P, t)); r.step(cfg.lr, cfg.eta)
        outs.append(r.state()); norms.append(r.grad_norms())
    for o, n in zip(outs[1:], norms[1:]):
        assert n == norms[0]
        for k in outs[0]:
            assert np.array_equal(outs[0][k], o[k]), k


def test_all_workers_pull_needs_no_norm_pass():
    cfg = _cfg(p=1.0)
    r = GpuRun(cfg, _x0(4, 5000), numel=[5000])
    r.set_grad_clip(0.1)
    r.set_grads(_grads(cfg, 5000, 0)); r.inner_step(cfg.lr, cfg.eta)
    assert r.lib.get_launch_count() == 2
    ss, cl = r.grad_norms()
    assert ss == [0.0] * 4 and cl == [1.0] * 4


def test_bad_thresholds_are_rejected():
    r = GpuRun(_cfg(), _x0(4, 64), numel=[64])
    for bad in (-1.0, float("nan"), float("inf")):
        with pytest.raises(Exception):
            r.set_grad_clip(bad)


@pytest.mark.parametrize("name,n_ddp", [("c3_gptneo125m_bf16", 0), ("c3_gptneo125m_bf16", 2), ("c2_resnet50", 1)])
def test_full_size_clipped_steps_sampled(name, n_ddp):
    """Benchmark-sized tensor lists: the oracle takes the exact sums of squares over the WHOLE
    gradients (copied back from the device) and replays a sample of indices with them."""
    cfg = W.get_config(name).with_(H=3)
    T = 4
    dev = torch.device("cuda:0")
    P = cfg.P
    idx = W.sample_indices(cfg.tensors, 1 << 13, seed=77)
    idx_d = torch.from_numpy(idx).to(dev)
    x_init = W.init_params_host(cfg.tensors, cfg.param_seed, cfg.init_std)
    gpu = GpuRun(cfg, np.broadcast_to(x_init, (cfg.K, P)))
    orc = make_oracle(cfg, np.tile(x_init[idx], (cfg.K, 1)))
    max_norm = 0.5 * cfg.grad_std * np.sqrt(P) / (np.sqrt(cfg.K) if n_ddp else 1.0)
    gpu.set_grad_clip(max_norm); orc.set_grad_clip(max_norm)
    gen = torch.Generator(device=dev); gen.manual_seed(cfg.grad_seed)
    grad_rows = gpu.arena["grad"][:, gpu.off:gpu.off + P]
    for t in range(T):
        scale = cfg.grad_std * (1.0 if t % 2 == 0 else 0.2)          # clipped / not clipped
        for k in range(cfg.K):
            grad_rows[k].copy_(torch.randn(P, generator=gen, device=dev, dtype=torch.float32).mul_(scale))
        full = grad_rows.contiguous()
        full = full.view(torch.int16).cpu().numpy().view(np.uint16) if cfg.precision == 1 else full.cpu().numpy()
        gs = full[:, idx]
        if t < n_ddp:                                                # norm of the averaged gradient, formed in fp32
            wide = (full.astype(np.uint32) << 16).view(np.float32) if cfg.precision == 1 else full
            gbar = wide[0].copy()
            for k in range(1, cfg.K):
                gbar += wide[k]
            gbar /= np.float32(cfg.K)
            orc.force_sumsq([oracle.sumsq(gbar)] * cfg.K)
            gpu.ddp_step(cfg.lr); orc.ddp_step(gs, cfg.lr)
            took = range(cfg.K)
        else:
            b = [oracle.decision(cfg.decision_seed, t, k, cfg.p) for k in range(cfg.K)]
            orc.force_sumsq([0.0 if b[k] else oracle.sumsq(full[k]) for k in range(cfg.K)])
            gpu.step(cfg.lr, cfg.eta); orc.step(gs, cfg.lr, cfg.eta)
            took = [k for k in range(cfg.K) if not b[k]]
        _check_norms(gpu, orc, took)
    got = {}
    for key, name_ in {"x": "master" if cfg.precision == 1 else "param", "m": "m", "v": "v", "xw": "param"}.items():
        if name_ in gpu.arena and not (key == "xw" and cfg.precision == 0):
            a = gpu.arena[name_][:, gpu.off:gpu.off + P][:, idx_d].contiguous()
            got[key] = a.view(torch.int16).cpu().numpy().view(np.uint16) if a.dtype == torch.bfloat16 else a.cpu().numpy()
    got["xg"] = gpu.arena["global_"][0, gpu.off:gpu.off + P][idx_d].cpu().numpy()
    got["u"] = gpu.arena["outer_mom"][0, gpu.off:gpu.off + P][idx_d].cpu().numpy()
    compare_state(got, orc, exact=True)
    assert gpu.guards_intact()
