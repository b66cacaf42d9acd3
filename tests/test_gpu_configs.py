"""GPU parity on the benchmark configurations.

Tier A (every element, host-generated gradients): the tiny flat run in full,
and the GPT-Neo-8M / ResNet-50 shaped lists over a shortened schedule.
Tier B (full size, full schedule, the launch configuration the benchmark times):
gradients are drawn on the device by torch's seeded generator (a harness input,
not the library); because the path is elementwise and the decisions depend only
on (seed, t, k), the oracle replays a sample of indices exactly -- every
tensor's first and last elements plus random positions -- and properties that
hold at any size (consensus after a sync, counters) are checked on everything.
"""
import numpy as np
import pytest
import torch

import workloads as W
from _harness import GpuRun, compare_state, make_oracle

pytestmark = pytest.mark.gpu


def _host_grads(cfg, P, t):
    g = np.stack([W.grads_host(P, cfg.grad_seed, t, k, cfg.grad_std) for k in range(cfg.K)])
    return W.bf16_bits_from_f32_host(g) if cfg.precision == 1 else g


def test_c0_tiny_flat_run_every_element_every_step():
    cfg = W.get_config("c0_flat_1m")
    P = cfg.P
    x0 = np.tile(W.init_params_host(cfg.tensors, cfg.param_seed, cfg.init_std), (cfg.K, 1))
    gpu, orc = GpuRun(cfg, x0), make_oracle(cfg, x0)
    for t in range(cfg.T):
        g = _host_grads(cfg, P, t)
        gpu.set_grads(g); gpu.step(cfg.lr, cfg.eta); orc.step(g, cfg.lr, cfg.eta)
        c = gpu.counters()
        assert c["last_b"] == [int(v) for v in orc.last_b] and c["s"] == [int(v) for v in orc.s]
    rep = compare_state(gpu.state(), orc, exact=True)
    assert gpu.counters()["n_outer"] == 2 and gpu.guards_intact()
    print("c0 parity", rep)


@pytest.mark.parametrize("name,layout", [("c1_gptneo8m", "arena"), ("c2_resnet50", "separate"),
                                         ("c2_resnet50", "arena")])
def test_model_shaped_lists_every_element_short_schedule(name, layout):
    cfg = W.get_config(name).with_(H=3, T=7, K=4)
    P = cfg.P
    x0 = np.tile(W.init_params_host(cfg.tensors, cfg.param_seed, cfg.init_std), (cfg.K, 1))
    gpu, orc = GpuRun(cfg, x0, layout=layout), make_oracle(cfg, x0)
    for t in range(cfg.T):
        g = _host_grads(cfg, P, t)
        gpu.set_grads(g); gpu.step(cfg.lr, cfg.eta); orc.step(g, cfg.lr, cfg.eta)
    compare_state(gpu.state(), orc, exact=True)
    c = gpu.counters()
    assert c["t"] == cfg.T and c["n_outer"] == cfg.T // cfg.H and c["s"] == [int(v) for v in orc.s]
    assert gpu.guards_intact()


def _full_size_sampled(cfg, n_random, T=None, n_ddp=0):
    """n_ddp: that many leading steps are DDP warm-up steps."""
    T = cfg.T if T is None else T
    dev = torch.device("cuda:0")
    tensors = cfg.tensors
    P = cfg.P
    idx = W.sample_indices(tensors, n_random, seed=99)
    idx_d = torch.from_numpy(idx).to(dev)
    x_init = W.init_params_host(tensors, cfg.param_seed, cfg.init_std)
    gpu = GpuRun(cfg, np.broadcast_to(x_init, (cfg.K, P)))
    orc = make_oracle(cfg, np.tile(x_init[idx], (cfg.K, 1)))
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.grad_seed)
    grad_rows = gpu.arena["grad"][:, gpu.off:gpu.off + P]
    for t in range(T):
        for k in range(cfg.K):                        # harness generator, one worker at a time
            r = torch.randn(P, generator=gen, device=dev, dtype=torch.float32).mul_(cfg.grad_std)
            grad_rows[k].copy_(r)                     # rounds to bf16 in mixed-precision mode
        gs = grad_rows[:, idx_d].contiguous()
        gs = gs.view(torch.int16).cpu().numpy().view(np.uint16) if cfg.precision == 1 else gs.cpu().numpy()
        if t < n_ddp:
            gpu.ddp_step(cfg.lr)
            orc.ddp_step(gs, cfg.lr)
        else:
            gpu.step(cfg.lr, cfg.eta)
            orc.step(gs, cfg.lr, cfg.eta)
    torch.cuda.synchronize()
    c = gpu.counters()
    assert c["t"] == orc.t == T and c["n_outer"] == orc.n_outer
    assert c["s"] == [int(v) for v in orc.s] and c["last_b"] == [int(v) for v in orc.last_b]
    names = {"x": "master" if cfg.precision == 1 else "param", "m": "m", "v": "v", "xw": "param"}
    got = {}
    for key, name in names.items():
        if name in gpu.arena and not (key == "xw" and cfg.precision == 0) and not (key == "x" and False):
            a = gpu.arena[name][:, gpu.off:gpu.off + P][:, idx_d].contiguous()
            got[key] = a.view(torch.int16).cpu().numpy().view(np.uint16) if a.dtype == torch.bfloat16 else a.cpu().numpy()
    got["xg"] = gpu.arena["global_"][0, gpu.off:gpu.off + P][idx_d].cpu().numpy()
    got["u"] = gpu.arena["outer_mom"][0, gpu.off:gpu.off + P][idx_d].cpu().numpy()
    rep = compare_state(got, orc, exact=True)
    # properties that hold at any size
    if T % cfg.H == 0:
        xg = gpu.arena["global_"][0, gpu.off:gpu.off + P]
        xf = gpu.arena["master" if cfg.precision == 1 else "param"][:, gpu.off:gpu.off + P]
        assert bool((xf == xg[None]).all())           # every slot restarted from the global model
        if cfg.precision == 1:
            w = gpu.arena["param"][:, gpu.off:gpu.off + P]
            assert bool((w == xg.to(torch.bfloat16)[None]).all())
    assert gpu.guards_intact()
    print(cfg.name, "sampled parity over", idx.size, "indices:", rep)


def test_c1_gptneo8m_full_size_full_schedule_sampled():
    _full_size_sampled(W.get_config("c1_gptneo8m"), 1 << 15)


def test_c2_resnet50_full_size_full_schedule_sampled():
    _full_size_sampled(W.get_config("c2_resnet50"), 1 << 15)


def test_c3_gptneo125m_bf16_full_size_full_schedule_sampled():
    _full_size_sampled(W.get_config("c3_gptneo125m_bf16"), 1 << 15)


def test_sweep_corner_k32_large_flat_buffer_sampled():
    cfg = next(c for c in W.sweep_points() if c.K == 32 and c.P == 1 << 24 and c.p == 0.5 and c.H == 16)
    _full_size_sampled(cfg, 1 << 14, T=32)


@pytest.mark.parametrize("name", ["c2_resnet50", "c3_gptneo125m_bf16"])
def test_ddp_warm_up_then_palsgd_full_size_sampled(name):
    cfg = W.get_config(name).with_(H=4)
    _full_size_sampled(cfg, 1 << 14, T=12, n_ddp=6)
