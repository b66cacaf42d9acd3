"""The controller of the several-GPU deployment (paper_2504_18454_b200/workers.py) on CPU: two gloo
ranks, each holding half of the workers, with a stand-in context whose arithmetic is the CPU
oracle's (per-worker steps with the job-wide decisions, the sum over local workers, and the
OuterOPT update) and the process group's all-reduce as the exchange.  Checked: which workers a
rank owns, that the local workers draw the job's decisions, when the synchronisation runs, that
both ranks end with the same global model, and that it agrees with ONE oracle holding all K workers
within the parity tolerance (the sum over k is grouped by rank, so rounding may differ)."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest

from paper_2504_18454_b200.workers import worker_span

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_worker_span_partitions_the_workers():
    assert [worker_span(8, r, 4) for r in range(4)] == [(0, 2), (2, 4), (4, 6), (6, 8)]
    assert worker_span(5, 0, 1) == (0, 5)
    with pytest.raises(ValueError):
        worker_span(6, 0, 4)
    with pytest.raises(ValueError):
        worker_span(8, 4, 4)


WORKER = r'''
import json, os, sys
sys.path.insert(0, sys.argv[1])
import numpy as np
import torch
import torch.distributed as dist
import oracle
import workloads as W
from paper_2504_18454_b200.workers import DistributedPalsgd, worker_span

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
K_total, P, H, T, p, seed = 4, 3001, 3, 7, 0.4, 77
lr, eta = 1e-3, 16.0
x_all = np.stack([W.init_params_host(W.flat_shape(P), 1234 + k, 0.02) for k in range(K_total)])    # workers start apart


class OracleContext:
    """Stands in for a device context: same methods, the oracle's arithmetic."""
    def __init__(self, K, exchange, k_first, x_start=None):
        self.K, self.H, self.exchange, self.k0 = K, H, exchange, None
        x_start = x_all if x_start is None else x_start
        self.orc = oracle.Oracle(x_start[k_first:k_first + K], K=K, H=10**9, p=p, seed=seed)
        self.calls = []
    def exchange_numel(self):
        return P
    def set_worker_offset(self, k0):
        self.k0 = k0
    def inner_step(self, lr_t, eta_t, stream=0):
        t = self.orc.t
        g = np.stack([W.grads_host(P, 5678, t, self.k0 + k, 0.01) for k in range(self.K)])
        forced = [oracle.decision(seed, t, self.k0 + k, p) for k in range(self.K)]
        self.orc.inner_step(g, lr_t, eta_t, forced=forced)
        self.calls.append("inner")
    def ddp_partial(self, ptr, stream=0):
        assert ptr == self.exchange.data_ptr()
        acc = W.grads_host(P, 5678, self.orc.t, self.k0, 0.01)
        for k in range(1, self.K):
            acc = acc + W.grads_host(P, 5678, self.orc.t, self.k0 + k, 0.01)   # float32, ascending local index
        self.exchange.copy_(torch.from_numpy(acc))
        self.calls.append("ddp_partial")
    def ddp_finish(self, ptr, K_tot, lr_t, stream=0):
        assert self.K == 2                                   # (gbar + gbar) / 2 is gbar exactly
        gbar = (self.exchange.numpy() / np.float32(K_tot)).astype(np.float32)
        self.orc.ddp_step(np.tile(gbar, (self.K, 1)), lr_t)
        self.calls.append("ddp_finish")
    def outer_partial(self, ptr, stream=0):
        assert ptr == self.exchange.data_ptr()
        acc = self.orc.x[0].copy()
        for k in range(1, self.K):
            acc = acc + self.orc.x[k]                       # float32, ascending local index
        self.exchange.copy_(torch.from_numpy(acc))
        self.calls.append("partial")
    def global_from_exchange(self, ptr, K_tot, stream=0):
        self.orc.xg[:] = (self.exchange.numpy() / np.float32(K_tot)).astype(np.float32)
        self.calls.append("global")
    def outer_finish(self, ptr, K_tot, stream=0):
        xbar = (self.exchange.numpy() / np.float32(K_tot)).astype(np.float32)
        one = oracle.Oracle(xbar[None], K=1, H=1, p=0.0)    # OuterOPT on a one-worker average = xbar
        one.xg[:] = self.orc.xg; one.u[:] = self.orc.u
        one.outer_sync()
        self.orc.xg[:] = one.xg; self.orc.u[:] = one.u
        self.orc.x[:] = one.xg[None]
        self.calls.append("finish")


k0, k1 = worker_span(K_total, rank, world)
exch = torch.zeros(P, dtype=torch.float32)
ctx = OracleContext(k1 - k0, exch, k0)
job = DistributedPalsgd(ctx, exch, K_total, rank, world)
job.init_global()
synced = [job.step(lr, eta) for _ in range(T)]

# the DDP warm-up phase: all workers start from one model; every rank must take the step of the job's mean gradient
x_same = np.tile(x_all[0], (K_total, 1))
exch2 = torch.zeros(P, dtype=torch.float32)
ctx2 = OracleContext(k1 - k0, exch2, k0, x_same)
job2 = DistributedPalsgd(ctx2, exch2, K_total, rank, world)
ddp_ref = oracle.Oracle(x_same, K=K_total, H=H, p=p, seed=seed, sum_groups=world)
for t in range(2):
    job2.ddp_step(lr)
    ddp_ref.ddp_step(np.stack([W.grads_host(P, 5678, t, k, 0.01) for k in range(K_total)]), lr)
ddp_ok = bool(job2.t == 2 and np.array_equal(ctx2.orc.x, ddp_ref.x[k0:k1]) and np.array_equal(ctx2.orc.m, ddp_ref.m[k0:k1])
              and np.array_equal(ctx2.orc.xg, ddp_ref.xg) and not np.array_equal(ddp_ref.xg, x_all[0]))

# one oracle with all the workers, ascending order over all k
ref = oracle.Oracle(x_all, K=K_total, H=H, p=p, seed=seed)
grouped = oracle.Oracle(x_all, K=K_total, H=H, p=p, seed=seed, sum_groups=world)   # sums as the two ranks form them
for t in range(T):
    g = np.stack([W.grads_host(P, 5678, t, k, 0.01) for k in range(K_total)])
    grouped.step(g, lr, eta)
for t in range(T):
    g = np.stack([W.grads_host(P, 5678, t, k, 0.01) for k in range(K_total)])
    ref.step(g, lr, eta)

gathered = [torch.zeros(P) for _ in range(world)]
dist.all_gather(gathered, torch.from_numpy(ctx.orc.xg.copy()))
err = lambda a, b: float(np.max(np.abs(a.astype(np.float64) - b) / np.maximum(np.abs(b), 1e-7 / 1e-6)))
out = {"rank": rank, "k0": ctx.k0, "synced": synced, "calls": ctx.calls,
       "same_xg_on_all_ranks": all(bool(torch.equal(gathered[0], g_)) for g_ in gathered),
       "s_equal": [int(v) for v in ctx.orc.s] == [int(v) for v in ref.s[k0:k1]],
       "err_xg": err(ctx.orc.xg, ref.xg), "err_u": err(ctx.orc.u, ref.u),
       "err_x": err(ctx.orc.x, ref.x[k0:k1]), "m_equal": bool(np.array_equal(ctx.orc.m, ref.m[k0:k1])),
       "ddp_ok": ddp_ok, "ddp_calls": ctx2.calls,
       "n_pulls": int(sum(T - int(v) for v in ref.s)),
       "bitwise_vs_grouped": bool(np.array_equal(ctx.orc.xg, grouped.xg) and np.array_equal(ctx.orc.u, grouped.u)
                                  and np.array_equal(ctx.orc.x, grouped.x[k0:k1]))}
with open(os.path.join(sys.argv[2], f"rank{rank}.json"), "w") as f:
    json.dump(out, f)
dist.barrier()
dist.destroy_process_group()
'''


def test_two_ranks_hold_half_of_the_workers_each(tmp_path):
    from conftest import free_port
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), str(script), ROOT, str(tmp_path)]
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-3000:]
    for rank in (0, 1):
        d = json.load(open(tmp_path / f"rank{rank}.json"))
        assert d["k0"] == 2 * rank
        assert d["synced"] == [False, False, True, False, False, True, False]       # H = 3, T = 7
        assert d["calls"] == (["partial", "global"] + ["inner"] * 3 + ["partial", "finish"] + ["inner"] * 3 +
                              ["partial", "finish"] + ["inner"])
        assert d["same_xg_on_all_ranks"] and d["s_equal"] and d["m_equal"] and d["bitwise_vs_grouped"]
        assert d["ddp_ok"] and d["ddp_calls"] == ["ddp_partial", "ddp_finish"] * 2
        assert 0 < d["n_pulls"] < 4 * 7                                           # both branches were taken
        for key in ("err_xg", "err_u", "err_x"):                                  # the parity bar: 1e-6 rel, 1e-7 abs floor
            assert d[key] <= 1e-6, (key, d[key])
