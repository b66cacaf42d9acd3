"""One packed tensor list of more than 2^32 elements per worker (a multi-billion-parameter model held as one
segment): element offsets no longer fit 32 bits anywhere on the path.  K = 1 and momentum SGD keep the state at
5 buffers x 17 GB; the oracle replays sampled indices (the path is elementwise), chosen around the places where a
32-bit offset would wrap, and properties that hold for every element are checked on the whole buffers."""
import gc

import numpy as np
import pytest
import torch

import oracle
import paper_2504_18454_b200 as P
import workloads as W
from paper_2504_18454_b200.arena import ReplicaArena
from _harness import compare_state

pytestmark = pytest.mark.gpu

N = (1 << 32) + 3 * 4096 + 5          # elements; the tail is ragged


@pytest.fixture(autouse=True)
def _give_the_memory_back():
    yield
    gc.collect(); torch.cuda.empty_cache()


def _indices():
    edges = [0, 8191, 8192, (1 << 31) - 1, 1 << 31, (1 << 32) - 8192, (1 << 32) - 1, 1 << 32, (1 << 32) + 8191,
             (1 << 32) + 8192, N - 5, N - 4, N - 1]
    near = np.concatenate([np.arange(e - 3, e + 4) for e in edges])
    rnd = np.random.default_rng(7).integers(0, N, size=4096)
    idx = np.unique(np.concatenate([near, rnd]))
    return idx[(idx >= 0) & (idx < N)].astype(np.int64)


def _bits(a: torch.Tensor) -> np.ndarray:
    a = a.contiguous()
    return a.view(torch.int16).cpu().numpy().view(np.uint16) if a.dtype == torch.bfloat16 else a.cpu().numpy()


@pytest.mark.parametrize("inner,precision", [(P.INNER_SGDM, P.PREC_FP32), (P.INNER_ADAMW, P.PREC_BF16_MASTER)])
def test_offsets_beyond_32_bits(inner, precision):
    bf, adam = precision == P.PREC_BF16_MASTER, inner == P.INNER_ADAMW
    # param + grad, m (+ v) (+ master), x, u, the exchange buffer, working room
    need = ((4 if bf else 8) + 4 + (4 if adam else 0) + (4 if bf else 0) + 8 + 4) * N + (8 << 30)
    gc.collect(); torch.cuda.empty_cache()                                  # what an earlier test's allocator cache holds
    free, _ = torch.cuda.mem_get_info()
    if free < need:
        pytest.skip(f"needs {need >> 30} GB of free device memory, {free >> 30} GB are free")
    dev = torch.device("cuda:0")
    K, H, p, lr, eta, seed = 1, 2, 0.5, 0.05, 2.0, 11
    arena = ReplicaArena([N], K, precision=precision, inner=inner, device=dev)
    gen = torch.Generator(device=dev); gen.manual_seed(1234)
    arena.model[0].normal_(0.0, 0.02, generator=gen)
    idx = _indices(); idx_d = torch.from_numpy(idx).to(dev)
    x0 = arena.model[:, idx_d].cpu().numpy()
    stream = torch.cuda.current_stream().cuda_stream
    hyper = dict(H=H, p=p, momentum=0.9 if not adam else 0.0, weight_decay=1e-4, outer_lr=0.7, outer_momentum=0.9,
                 outer_nesterov=True, seed=seed)
    ctx = arena.make_context(stream=stream, **hyper)
    orc = oracle.Oracle(x0, K=K, inner=inner, precision=precision, **hyper)
    assert ctx.get_layout() == {"n_segments": 1, "n_chunks": -(-N // 8192), "chunk_elems": 8192}
    assert torch.equal(arena.rows("global_")[0], arena.model[0])           # init: the mean of one slot is the slot
    grad = arena.rows("grad")[0]
    exch = torch.zeros(ctx.exchange_numel(), dtype=torch.float32, device=dev)
    assert exch.numel() >= N

    def gradients():
        grad.normal_(0.0, 0.01, generator=gen)              # (rounds to bf16 in mixed-precision mode)
        return _bits(grad[idx_d])[None]

    g = gradients()
    ctx.ddp_step(lr, stream); orc.ddp_step(g, lr)                          # t = 0: a DDP warm-up step
    g = gradients()                                                         # t = 1: one in its several-GPU form
    ctx.ddp_partial(exch.data_ptr(), stream); ctx.ddp_finish(exch.data_ptr(), K, lr, stream); orc.ddp_step(g, lr)
    decisions = []
    for t in range(2, 8):
        g = gradients()
        orc.inner_step(g, lr, eta)
        ctx.inner_step(lr, eta, stream)
        decisions.append(int(orc.last_b[0]))
        if (t + 1) % H == 0:
            orc.outer_sync()
            if t == 3:
                ctx.outer_sync(stream)
            else:                                                           # the several-GPU form, one rank
                ctx.outer_partial(exch.data_ptr(), stream)
                ctx.outer_finish(exch.data_ptr(), K, stream)
            assert torch.equal(arena.model[0], arena.rows("global_")[0])    # every element restarted from x
    assert 0 < sum(decisions) < len(decisions)                              # both branches were taken
    c = ctx.get_counters(stream)
    assert c["t"] == orc.t == 8 and c["n_outer"] == orc.n_outer == 3 and c["s"] == [int(v) for v in orc.s]
    got = {"x": arena.model[:, idx_d].cpu().numpy(), "m": arena.rows("m")[:, idx_d].cpu().numpy(),
           "xg": arena.rows("global_")[0][idx_d].cpu().numpy(), "u": arena.rows("outer_mom")[0][idx_d].cpu().numpy()}
    if adam:
        got["v"] = arena.rows("v")[:, idx_d].cpu().numpy()
    if bf:
        got["xw"] = _bits(arena.rows("param")[:, idx_d])
    compare_state(got, orc, exact=True)

    # the norm pass over every element: a constant gradient whose sum of squares is exact by hand
    grad.fill_(0.5)
    ctx.set_grad_clip(1.0)
    while P.decision(seed, ctx.get_counters(stream)["t"], 0, p):            # a step on which the worker takes a gradient
        ctx.inner_step(lr, eta, stream)
    ctx.inner_step(lr, eta, stream)
    sumsq, clip = ctx.get_grad_norms(stream)
    assert sumsq[0] == N * 0.25                                             # exactly representable (0.5 is a bf16 value)
    assert np.float32(clip[0]) == np.float32(oracle.clip_coef(N * 0.25, 1.0))
