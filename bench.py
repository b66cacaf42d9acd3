#!/usr/bin/env python
"""Benchmark of the PALSGD update / synchronisation path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A "step" is one iteration of Algorithm 1 for all K workers: the fused inner
kernel (branch draw + optimizer step or pull), plus the outer-sync kernel on
every H-th step.  The metric is worker-element updates per second (K*P per
step), whole job.  Inputs are synthetic (model-shaped buffers, seeded normal
values) and resident in device memory before the timed region; the `e2e` figure
repeats the measurement through palsgd_step_host with gradients in pinned host
memory and results read back to the host every step.

With N > 1 (launched by torch.distributed.run) every rank runs an independent
replica of the workload on its own GPU: the path has no cross-GPU exchange.
One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import workloads as W  # noqa: E402

METRIC = "param_updates_per_s"
UNIT = "worker-element updates/s"
DEFAULT_WORKLOAD = "c3_gptneo125m_bf16"


# ----------------------------------------------------------------------------- helpers

def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


# DRAM traffic (ncu: dram__bytes_read.sum + dram__bytes_write.sum) divided by the algorithmic bytes
# of the same launch, measured on the 16M-element stand-ins of the same kernels (all-gradient inner
# launch; outer launch).  Traffic grows in proportion to the elements processed, so the ratio carries
# over to the full-size launch.  Valid only for the kernel sources with the digest recorded here.
NCU_TRAFFIC = {"digest": "863f86b42b326612",
               "inner": {0: 0.990, 1: 0.985},      # by precision: fp32, bf16 + fp32 master
               "outer": {0: 0.957, 1: 0.963},
               "ddp": {0: 0.976, 1: 0.975}}


def kernel_digest() -> str:
    import hashlib
    h = hashlib.sha256()
    for f in ("palsgd_device.cuh", "palsgd_kernels.cuh"):
        with open(os.path.join(ROOT, "paper_2504_18454_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(kind: str, precision: int, alg_bytes_per_launch):
    """Measured DRAM bytes per launch, or None once the kernels changed since the capture."""
    if alg_bytes_per_launch is None or kernel_digest() != NCU_TRAFFIC["digest"]:
        return None
    return NCU_TRAFFIC[kind][precision] * alg_bytes_per_launch


def inner_bytes_per_element(cfg, pull: bool) -> int:
    """Algorithmic HBM bytes per worker-element of the fused inner kernel."""
    bf = cfg.precision == 1
    if pull:                       # read x, x_g; write x (+ bf16 working copy)
        return 14 if bf else 12
    if cfg.inner == 0:             # AdamW: read g, x, m, v; write x, m, v (+ bf16 copy; bf16 g)
        return 28
    return 18 if bf else 20        # momentum SGD: read g, x, buf; write x, buf


def ddp_bytes_per_param(cfg) -> int:
    """DDP warm-up step: read K gradients and worker 0's x, m(, v); write x, m(, v) of all K slots
    (+ K bf16 working copies) and x_g.  16K+16 (AdamW) or 12K+12 (momentum SGD) in both precisions."""
    return (16 if cfg.inner == 0 else 12) * (cfg.K + 1)


def outer_bytes_per_param(cfg) -> int:
    """Read K slots, x_g, u; write x_g, u, K slots (+ K bf16 working copies)."""
    return (10 if cfg.precision == 1 else 8) * cfg.K + 16


def max_over_ranks(values, world: int, device=None):
    """Element-wise MAX of a list of floats over all ranks (the timing rule for N > 1: a job is as
    slow as its slowest rank).  With one rank the list comes back unchanged."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_value(world: int, K: int, P: int, steps: int, ms_total: float) -> float:
    """Worker-element updates per second of the whole job: every rank updates K*P elements per step."""
    return world * K * P * steps / (ms_total * 1e-3)


def rank_share(numel, rank: int, world: int, shard: bool):
    """What one rank of the job holds.  Replicas (default): the whole tensor list, a model of its own
    (seed offset = rank), so the job updates world * P elements per worker and step (weak scaling).
    Shards: its slice [lo, hi) of the parameter axis of ONE model (seed offset 0), so the job updates P
    elements per worker and step however many ranks there are (strong scaling).
    Returns (numel of the rank's tensor list, lo, hi, seed offset, elements per worker of the whole job)."""
    P = int(sum(numel))
    if not shard:
        return [int(n) for n in numel], 0, P, rank, P * world
    from paper_2504_18454_b200.shard import shard_numel, shard_span
    lo, hi = shard_span(numel, rank, world)
    mine = shard_numel(numel, rank, world)
    assert hi - lo == sum(mine)
    return mine, lo, hi, 0, P


class ClockSampler:
    """nvidia-smi clock / throttle sampling while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()                      # the exact process started above
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2])); pw.append(float(f[3]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                      "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        finally:
            try:
                os.unlink(self.path)
            except OSError:
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- CPU oracle leg

def time_oracle(cfg, steps: int, P_sample: int, H: int, threads: int = 0):
    """The CPU oracle, as it stands, on the first P_sample elements of the workload
    (threads = 0: every core the process may use)."""
    import oracle
    all_threads = oracle.get_threads()
    if threads:
        oracle.set_threads(threads)
    try:
        return _time_oracle(cfg, steps, P_sample, H)
    finally:
        oracle.set_threads(all_threads)


def _time_oracle(cfg, steps: int, P_sample: int, H: int):
    import oracle
    K = cfg.K
    x_init = W.init_params_host(W.flat_shape(P_sample), cfg.param_seed, cfg.init_std)
    o = oracle.Oracle(np.tile(x_init, (K, 1)), dtype="f32", K=K, H=H, p=cfg.p, inner=cfg.inner,
                      beta1=cfg.beta1, beta2=cfg.beta2, eps=cfg.eps, weight_decay=cfg.weight_decay,
                      momentum=cfg.momentum, outer_lr=cfg.outer_lr, outer_momentum=cfg.outer_momentum,
                      outer_nesterov=cfg.outer_nesterov, seed=cfg.decision_seed, precision=cfg.precision)
    g = np.stack([W.grads_host(P_sample, cfg.grad_seed, 0, k, cfg.grad_std) for k in range(K)])
    if cfg.precision == 1:
        g = W.bf16_bits_from_f32_host(g)
    o.step(g, cfg.lr, cfg.eta)                     # warm the pages
    t0 = time.perf_counter()
    for _ in range(steps):
        o.step(g, cfg.lr, cfg.eta)
    dt = time.perf_counter() - t0
    return K * P_sample * steps / dt, dt, oracle.get_threads(), o.n_outer


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    P_sample = min(cfg.P, 1 << 21)
    H = cfg.H                                   # the workload's own interval, as printed in `config`
    for _ in range(max(args.warmup, 0)):
        time_oracle(cfg, 1, P_sample, H)
    value, dt, cores, n_outer = time_oracle(cfg, args.steps, P_sample, H)
    sample = (f"first {P_sample} of {cfg.P} elements per worker, K={cfg.K}, {args.steps} steps, "
              f"H={H} ({n_outer} outer syncs)")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": dtype_of(cfg),
        "data": "synthetic", "config": workload_config(cfg, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def dtype_of(cfg) -> str:
    """The arithmetic type of the path (every element operation is binary32), with the storage types
    of the mixed-precision workloads spelled out."""
    return "f32" if cfg.precision == 0 else "f32 arithmetic; bf16 params+grads, f32 master/moments"


def roofline_entry(kernel: str, kind: str, cfg, peak: float, peak_src: str, ms_sum: float, bytes_sum: float,
                   n: int, units_per_launch: int = 0, **extra) -> dict:
    """One roofline object: achieved = algorithmic bytes / CUDA-event time of the kernel's launches."""
    gbs = bytes_sum / (ms_sum * 1e-3) / 1e9 if ms_sum else None
    d = {"bound": "hbm", "kernel": kernel, "achieved": gbs, "peak": peak, "unit": "GB/s",
         "frac": gbs / peak if gbs else None,
         "traffic": ncu_traffic(kind, cfg.precision, bytes_sum / n if n else None),
         "peak_source": peak_src,
         "frac_of_measured_copy": gbs / peak if gbs else None,
         "frac_of_nominal_peak": gbs / 8000.0 if gbs else None, "nominal_peak": 8000.0,
         "launches": n, "avg_ms": ms_sum / n if n else None,
         "alg_bytes_per_launch": bytes_sum / n if n else None}
    if units_per_launch and ms_sum:
        d["params_per_s"] = units_per_launch * n / (ms_sum * 1e-3)
    d.update(extra)
    return d


def workload_config(cfg, args) -> dict:
    return {"workload": cfg.name, "K": cfg.K, "P": cfg.P, "n_tensors": len(cfg.tensors), "H": cfg.H,
            "layout": getattr(args, "layout", "arena"),
            "p": cfg.p, "eta": cfg.eta, "lr": cfg.lr,
            "inner": "adamw" if cfg.inner == 0 else "sgdm",
            "precision": "bf16 params+grads, fp32 master/moments" if cfg.precision == 1 else "fp32",
            "parallelism": (f"parameter-axis shards x{args.gpus}" if getattr(args, "shard", False)
                            else f"replicas x{args.gpus}") if args.gpus > 1 else "single GPU",
            "l2": "state far larger than L2 (no flush needed)"
                  if cfg.K * cfg.P * 16 > 4 * 126e6 else "L2-affected: state comparable to the 126 MB L2"}


# ----------------------------------------------------------------------------- GPU leg

def run_workers(args, cfg):
    """The deployment the paper runs: the K workers spread over the ranks (K / world each, one rank per GPU),
    inner steps local, every H steps the outer sync as local sum -> all-reduce(sum) over NCCL -> finish
    (Algorithm 1's All-Reduce).  Total work is fixed as the ranks grow ("strong").  One JSON line from rank 0."""
    import torch
    import torch.distributed as dist
    import paper_2504_18454_b200 as P
    from paper_2504_18454_b200.arena import ReplicaArena
    from paper_2504_18454_b200.workers import DistributedPalsgd, worker_span

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.gpus > 1 and world != args.gpus:
        raise SystemExit("launch with: python -m torch.distributed.run --nnodes=1 --nproc-per-node N "
                         "--master-addr 127.0.0.1 --master-port P bench.py --gpus N --workers ...")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if "RANK" in os.environ:                             # under torchrun, one rank included: the collective is NCCL's
        dist.init_process_group("nccl", device_id=dev)
    k0, k1 = worker_span(cfg.K, rank, world)
    K, Kl, Pn = cfg.K, k1 - k0, cfg.P
    numel = [t.numel for t in cfg.tensors]

    def barrier():
        if dist.is_initialized():
            dist.barrier()
        torch.cuda.synchronize(dev)

    arena = ReplicaArena(numel, Kl, precision=cfg.precision, inner=cfg.inner, device=dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.param_seed)                      # one initial model for the whole job (Algorithm 1)
    x0 = torch.randn(Pn, generator=gen, device=dev).mul_(cfg.init_std)
    for k in range(Kl):
        arena.write_flat(arena.model_name, k, x0)
        gen.manual_seed(cfg.grad_seed + k0 + k)          # one gradient per worker of the job
        arena.write_flat("grad", k, torch.randn(Pn, generator=gen, device=dev).mul_(cfg.grad_std))
    del x0
    stream = torch.cuda.current_stream(dev).cuda_stream
    ctx = arena.make_context(
        stream=stream, H=cfg.H, p=cfg.p, beta1=cfg.beta1, beta2=cfg.beta2, eps=cfg.eps, weight_decay=cfg.weight_decay,
        momentum=cfg.momentum, outer_lr=cfg.outer_lr, outer_momentum=cfg.outer_momentum,
        outer_nesterov=cfg.outer_nesterov, seed=cfg.decision_seed)
    exch = torch.zeros(ctx.exchange_numel(), dtype=torch.float32, device=dev)

    def all_reduce_sum(buf):
        if dist.is_initialized():
            dist.all_reduce(buf, op=dist.ReduceOp.SUM)   # on torch's current stream, the one the kernels use

    job = DistributedPalsgd(ctx, exch, K, rank, world, all_reduce_sum=all_reduce_sum)
    job.init_global(stream)

    def one_step(rec=None):
        ev = lambda: torch.cuda.Event(enable_timing=True)
        e = [ev() for _ in range(5)]
        e[0].record(); job.inner_step(cfg.lr, cfg.eta, stream); e[1].record()       # (counts the step in job.t)
        if job.t % cfg.H == 0:
            ctx.outer_partial(exch.data_ptr(), stream); e[2].record()
            all_reduce_sum(exch); e[3].record()
            ctx.outer_finish(exch.data_ptr(), K, stream); e[4].record()
            if rec is not None:
                rec.append(("sync", job.t, e))
        elif rec is not None:
            rec.append(("inner", job.t, e))

    for _ in range(max(args.warmup, 3)):
        one_step()
    while job.t % cfg.H != 0:                            # the timed region starts right behind a synchronisation
        one_step()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = ctx.get_launch_count()
    rec = []
    barrier()
    e_start = torch.cuda.Event(enable_timing=True); e_end = torch.cuda.Event(enable_timing=True)
    e_start.record()
    for _ in range(args.steps):
        one_step(rec)
    e_end.record()
    barrier()
    ms_total = e_start.elapsed_time(e_end)
    launches = ctx.get_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None

    inner_ms = inner_bytes = part_ms = coll_ms = fin_ms = 0.0
    n_sync = 0
    for kind, t_after, e in rec:
        inner_ms += e[0].elapsed_time(e[1])
        inner_bytes += sum(inner_bytes_per_element(cfg, bool(P.decision(cfg.decision_seed, t_after - 1, k0 + k, cfg.p)))
                           for k in range(Kl)) * Pn
        if kind == "sync":
            part_ms += e[1].elapsed_time(e[2]); coll_ms += e[2].elapsed_time(e[3]); fin_ms += e[3].elapsed_time(e[4])
            n_sync += 1
    ms_total, inner_ms, part_ms, coll_ms, fin_ms = max_over_ranks([ms_total, inner_ms, part_ms, coll_ms, fin_ms], world, dev)
    if dist.is_initialized():
        dist.destroy_process_group()
    if rank != 0:
        return
    peak, peak_src = measured_peak_gbs()
    g_es = 2 if cfg.precision == 1 else 4
    sync_part = lambda name, ms, per_param: ({"kernel": name, "avg_ms": ms / n_sync,
                                              "achieved": per_param * Pn * n_sync / (ms * 1e-3) / 1e9, "unit": "GB/s"}
                                             if n_sync and ms > 0 else None)
    out = {
        "metric": METRIC, "value": K * Pn * args.steps / (ms_total * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_total / args.steps,
        "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": dtype_of(cfg), "data": "synthetic",
        "config": dict(workload_config(cfg, args), parallelism=f"{Kl} of the {K} workers per GPU; outer sync as local "
                       f"sum -> all-reduce(sum) of {Pn} floats -> finish every H steps"),
        "roofline": roofline_entry("palsgd_inner_kernel", "inner", cfg, peak, peak_src, inner_ms, inner_bytes, len(rec),
                                   units_per_launch=Kl * Pn, traffic=None),
        "outer_exchange": {"syncs": n_sync,
                           "partial": sync_part("palsgd_outer_partial_kernel", part_ms, 4 * Kl + 4),
                           "all_reduce": ({"avg_ms": coll_ms / n_sync, "bytes": 4 * Pn,
                                           "backend": "nccl" if world > 1 or "RANK" in os.environ else "none (one rank)"}
                                          if n_sync else None),
                           "finish": sync_part("palsgd_outer_kernel (sum from the exchange buffer)", fin_ms,
                                               (6 if cfg.precision == 1 else 4) * Kl + 20)},
        "cpu_baseline": None, "e2e": None, "gpu_launches": launches, "clocks": clocks,
        "note": "workers spread over the ranks; times are the maximum over ranks; gradients stay resident (no end-to-end "
                "leg in this mode)",
    }
    print(json.dumps(out), flush=True)


def run_ours(args, cfg):
    import torch
    import torch.distributed as dist
    import paper_2504_18454_b200 as P
    from paper_2504_18454_b200.arena import ReplicaArena

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.gpus > 1 and world != args.gpus:
        raise SystemExit("launch with: python -m torch.distributed.run --nnodes=1 --nproc-per-node N "
                         "--master-addr 127.0.0.1 --master-port P bench.py --gpus N ...")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    # CPU baseline first (rank 0, single-GPU runs only), before the GPU is busy
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # a bounded sample: about 10 s on all cores (step count found from a short trial), 3 s on one
        P_s = min(cfg.P, 1 << 21)
        rate, _, _, _ = time_oracle(cfg, 8, P_s, cfg.H)
        n_steps = int(max(16, min(8192, 10.0 * rate / (cfg.K * P_s))))
        value, dt, cores, n_outer = time_oracle(cfg, n_steps, P_s, cfg.H)
        P_1 = min(cfg.P, 1 << 18)
        rate1, _, _, _ = time_oracle(cfg, 4, P_1, cfg.H, threads=1)
        n_1 = int(max(8, min(8192, 3.0 * rate1 / (cfg.K * P_1))))
        value1, dt1, _, _ = time_oracle(cfg, n_1, P_1, cfg.H, threads=1)
        cpu_baseline = {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": f"first {P_s} of {cfg.P} elements per worker, K={cfg.K}, {n_steps} steps incl. "
                                  f"{n_outer} outer syncs (H={cfg.H}), {dt:.1f} s",
                        "single_thread_value": value1,
                        "single_thread_sample": f"first {P_1} elements per worker, {n_1} steps, {dt1:.1f} s"}

    # ---- buffers: seeded synthetic values, resident in HBM
    K = cfg.K
    # shards: every rank owns a slice of the parameter axis of all K slots of ONE model; the path is
    # elementwise and the decisions depend on (seed, t, k) only, so no exchange is needed
    numel, lo, hi, seed_off, P_job = rank_share([t.numel for t in cfg.tensors], rank, world, args.shard)
    Pn = hi - lo
    arena = ReplicaArena(numel, K, precision=cfg.precision, inner=cfg.inner, device=dev, layout=args.layout)
    x_full = W.init_params_host(cfg.tensors, cfg.param_seed + seed_off, cfg.init_std)
    x_init = torch.from_numpy(x_full[lo:lo + Pn]).to(dev)
    del x_full
    for k in range(K):
        arena.write_flat(arena.model_name, k, x_init)
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.grad_seed + rank)
    for k in range(K):
        arena.write_flat("grad", k, torch.randn(Pn, generator=gen, device=dev, dtype=torch.float32).mul_(cfg.grad_std))
    del x_init
    stream = torch.cuda.current_stream(dev).cuda_stream
    ctx = arena.make_context(
        stream=stream, H=cfg.H, p=cfg.p, beta1=cfg.beta1, beta2=cfg.beta2, eps=cfg.eps,
        weight_decay=cfg.weight_decay, momentum=cfg.momentum, outer_lr=cfg.outer_lr,
        outer_momentum=cfg.outer_momentum, outer_nesterov=cfg.outer_nesterov, seed=cfg.decision_seed)
    layout_info = ctx.get_layout()

    if args.inner_variant:
        ctx.set_tuning(P.TUNE_INNER_VARIANT, args.inner_variant)
    if args.grad_clip > 0:
        ctx.set_grad_clip(args.grad_clip)
    t_host = 0                                           # mirrors the library's step counter
    def one_step(ev_list=None):
        nonlocal t_host
        if ev_list is not None:
            e = torch.cuda.Event(enable_timing=True); e.record(); ev_list.append(("inner", t_host, e))
        ctx.inner_step(cfg.lr, cfg.eta, stream)
        t_host += 1
        if t_host % cfg.H == 0:
            if ev_list is not None:
                e = torch.cuda.Event(enable_timing=True); e.record(); ev_list.append(("outer", t_host, e))
            ctx.outer_sync(stream)

    for _ in range(max(args.warmup, 3)):
        one_step()
    # align the timed region so that it contains floor(steps / H) outer syncs in a fixed pattern
    while t_host % cfg.H != 0:
        one_step()

    # ---- timed region: device-resident inputs
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = ctx.get_launch_count()
    events = []
    barrier()
    e_start = torch.cuda.Event(enable_timing=True); e_end = torch.cuda.Event(enable_timing=True)
    e_start.record()
    for _ in range(args.steps):
        one_step(events)
    e_end.record()
    barrier()
    ms_total = e_start.elapsed_time(e_end)
    launches = ctx.get_launch_count() - launches0
    events.append(("end", t_host, e_end))

    # per-kernel durations (event to next event on the same stream) and algorithmic bytes
    inner_ms = inner_bytes = outer_ms = outer_bytes = 0.0
    n_inner = n_outer = 0
    for (kind, t_after, ev), (_, _, nxt) in zip(events[:-1], events[1:]):
        d = ev.elapsed_time(nxt)
        if kind == "inner":
            b = sum(inner_bytes_per_element(cfg, bool(P.decision(cfg.decision_seed, t_after, k, cfg.p)))
                    for k in range(K)) * Pn
            inner_ms += d; inner_bytes += b; n_inner += 1
        else:
            outer_ms += d; outer_bytes += outer_bytes_per_param(cfg) * Pn; n_outer += 1
    in_loop_outer = n_outer

    # ---- the outer-sync kernel on its own (the metric's "per outer_sync" half), whatever --steps is:
    # launches behind slots that two inner steps have let diverge again, one CUDA-event pair each,
    # under the same load (and clocks) as the step loop, which continues around them
    outer_alone = []
    if not args.no_outer:
        for i in range(args.outer_launches + 1):
            for _ in range(2):
                ctx.inner_step(cfg.lr, cfg.eta, stream); t_host += 1
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
            ctx.outer_sync(stream)
            e1.record()
            if i > 0:                                    # the first one is a warm-up
                outer_alone.append((e0, e1))
        torch.cuda.synchronize(dev)
        for e0, e1 in outer_alone:
            outer_ms += e0.elapsed_time(e1); outer_bytes += outer_bytes_per_param(cfg) * Pn; n_outer += 1
    clocks = sampler.stop() if rank == 0 else None

    # ---- end to end: gradients from pinned host memory, results back to the host, every step
    e2e = None
    if not args.no_e2e:
        gdt = torch.bfloat16 if cfg.precision == 1 else torch.float32
        h_grad = torch.empty((K, Pn), dtype=gdt).pin_memory()
        for k in range(K):
            h_grad[k].copy_(arena.read_flat("grad", k))
        h_glob = torch.empty(Pn, dtype=torch.float32).pin_memory()
        h_dec = torch.zeros(K, dtype=torch.uint8).pin_memory()
        es = h_grad.element_size()
        gp = ctx.make_ptr_array([h_grad.data_ptr() + (k * Pn + arena.starts[j]) * es
                                 for k in range(K) for j in range(len(numel))])
        xp = ctx.make_ptr_array([h_glob.data_ptr() + arena.starts[j] * 4 for j in range(len(numel))])
        e2e_steps = args.e2e_steps if args.e2e_steps > 0 else min(args.steps, cfg.H)
        for _ in range(2):
            ctx.step_host(gp, cfg.lr, cfg.eta, xp, h_dec.data_ptr(), stream); t_host += 1
        while t_host % cfg.H != (cfg.H - e2e_steps) % cfg.H:          # end the region on a sync step
            ctx.step_host(gp, cfg.lr, cfg.eta, xp, h_dec.data_ptr(), stream); t_host += 1
        barrier()
        s0 = torch.cuda.Event(enable_timing=True); s1 = torch.cuda.Event(enable_timing=True)
        s0.record()
        syncs = 0
        copied_workers = 0                                 # pulling workers' gradients are not transferred
        for _ in range(e2e_steps):
            copied_workers += sum(1 - P.decision(cfg.decision_seed, t_host, k, cfg.p) for k in range(K))
            syncs += int(ctx.step_host(gp, cfg.lr, cfg.eta, xp, h_dec.data_ptr(), stream)); t_host += 1
        s1.record()
        barrier()
        ms_e2e = s0.elapsed_time(s1)
        e2e = {"ms": ms_e2e, "steps": e2e_steps, "syncs": syncs,
               "h2d": copied_workers * Pn * es / e2e_steps, "d2h": K + syncs * Pn * 4 / e2e_steps}

    # ---- one H-step cycle as a single CUDA graph (launch overhead removed), timed on its own
    graph_cycle = None
    if not args.no_graph and args.grad_clip == 0:
        while t_host % cfg.H != 0:
            one_step()
        ctx.cycle_capture(cfg.lr, cfg.eta)
        n_cyc = max(1, min(64, int(0.5 / max(1e-6, (ms_total / args.steps) * 1e-3 * cfg.H))))
        ctx.cycle_launch(stream); t_host += cfg.H            # warm-up
        g0 = torch.cuda.Event(enable_timing=True); g1 = torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(n_cyc):
            ctx.cycle_launch(stream); t_host += cfg.H
        g1.record()
        torch.cuda.synchronize(dev)
        graph_cycle = {"cycles": n_cyc, "steps_per_cycle": cfg.H,
                       "ms_per_step": g0.elapsed_time(g1) / (n_cyc * cfg.H),
                       "value": K * Pn * n_cyc * cfg.H / (g0.elapsed_time(g1) * 1e-3), "unit": UNIT,
                       "note": "H inner launches + outer sync replayed as one CUDA graph; not part of value"}

    # ---- DDP warm-up kernel (the phase before Algorithm 1), timed on its own after the main regions
    ddp = None
    if not args.no_ddp:
        for _ in range(3):
            ctx.ddp_step(cfg.lr, stream)
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(9)]
        evs[0].record()
        for i in range(8):
            ctx.ddp_step(cfg.lr, stream)
            evs[i + 1].record()
        torch.cuda.synchronize(dev)
        ddp_ms = sum(evs[i].elapsed_time(evs[i + 1]) for i in range(8))
        ddp = {"ms": ddp_ms, "bytes": 8 * ddp_bytes_per_param(cfg) * Pn, "launches": 8}

    # ---- the outer sync split around an exchange buffer (the form for workers spread over several GPUs;
    # here one GPU, so the all-reduce between the two kernels is empty), timed on its own
    split = None
    if not args.no_ddp and world == 1:
        exch = torch.zeros(ctx.exchange_numel(), dtype=torch.float32, device=dev)
        pe, fe = [], []
        for i in range(5):
            for _ in range(2):
                ctx.inner_step(cfg.lr, cfg.eta, stream)
            e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            e0.record(); ctx.outer_partial(exch.data_ptr(), stream)
            e1.record(); ctx.outer_finish(exch.data_ptr(), K, stream)
            e2.record()
            if i > 0:
                pe.append((e0, e1)); fe.append((e1, e2))
        dpe, dfe = [], []                                  # the DDP warm-up step, split the same way
        g_es = 2 if cfg.precision == 1 else 4              # bytes per gradient element
        for i in range(5):
            e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            e0.record(); ctx.ddp_partial(exch.data_ptr(), stream)
            e1.record(); ctx.ddp_finish(exch.data_ptr(), K, cfg.lr, stream)
            e2.record()
            if i > 0:
                dpe.append((e0, e1)); dfe.append((e1, e2))
        torch.cuda.synchronize(dev)
        split = {"n": len(pe), "partial_ms": sum(a.elapsed_time(b) for a, b in pe),
                 "finish_ms": sum(a.elapsed_time(b) for a, b in fe),
                 "partial_bytes": len(pe) * (4 * K + 4) * Pn,
                 "finish_bytes": len(fe) * ((6 if cfg.precision == 1 else 4) * K + 20) * Pn,
                 "ddp_partial_ms": sum(a.elapsed_time(b) for a, b in dpe),
                 "ddp_finish_ms": sum(a.elapsed_time(b) for a, b in dfe),
                 "ddp_partial_bytes": len(dpe) * (g_es * K + 4) * Pn,
                 "ddp_finish_bytes": len(dfe) * (ddp_bytes_per_param(cfg) - g_es * K + 4) * Pn}
        del exch

    # ---- the same two kernels on a ragged device layout (one allocation per worker and tensor), timed on their
    # own after the main regions: frameworks hold their parameters that way, and the packed arenas above are
    # the friendliest case for the multi-tensor metadata
    ragged = None
    if args.layout == "arena" and world == 1 and not args.no_ragged and len(numel) > 1:
        arena2 = ReplicaArena(numel, K, precision=cfg.precision, inner=cfg.inner, device=dev, layout="separate")
        for k in range(K):
            arena2.write_flat(arena2.model_name, k, arena.read_flat(arena.model_name, k))
            arena2.write_flat("grad", k, arena.read_flat("grad", k))
        ctx2 = arena2.make_context(
            stream=stream, H=1 << 40, p=cfg.p, beta1=cfg.beta1, beta2=cfg.beta2, eps=cfg.eps,
            weight_decay=cfg.weight_decay, momentum=cfg.momentum, outer_lr=cfg.outer_lr,
            outer_momentum=cfg.outer_momentum, outer_nesterov=cfg.outer_nesterov, seed=cfg.decision_seed)
        n_in, n_out = 16, 4
        for _ in range(3):
            ctx2.inner_step(cfg.lr, cfg.eta, stream)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(n_in + 1)]
        ev[0].record()
        for i in range(n_in):
            ctx2.inner_step(cfg.lr, cfg.eta, stream); ev[i + 1].record()
        oev = []
        for i in range(n_out + 1):
            for _ in range(2):
                ctx2.inner_step(cfg.lr, cfg.eta, stream)
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record(); ctx2.outer_sync(stream); e1.record()
            if i > 0:
                oev.append((e0, e1))
        torch.cuda.synchronize(dev)
        in_ms = sum(ev[i].elapsed_time(ev[i + 1]) for i in range(n_in))
        in_bytes = sum(inner_bytes_per_element(cfg, bool(P.decision(cfg.decision_seed, 3 + i, k, cfg.p)))
                       for i in range(n_in) for k in range(K)) * Pn
        out_ms = sum(a.elapsed_time(b) for a, b in oev)
        ragged = {"layout": "separate", **ctx2.get_layout(), "inner_ms": in_ms, "inner_bytes": in_bytes, "n_inner": n_in,
                  "outer_ms": out_ms, "outer_bytes": n_out * outer_bytes_per_param(cfg) * Pn, "n_outer": n_out}
        ctx2.destroy()
        del ctx2, arena2

    # ---- max over ranks
    ms_total, ms_e2e_max = max_over_ranks([ms_total, e2e["ms"] if e2e else 0.0], world, dev)
    if e2e:
        e2e["ms"] = ms_e2e_max
    if rank == 0:
        peak, peak_src = measured_peak_gbs()
        value = whole_job_value(1, K, P_job, args.steps, ms_total)
        r_inner = roofline_entry("palsgd_inner_kernel", "inner", cfg, peak, peak_src, inner_ms, inner_bytes, n_inner)
        r_outer = roofline_entry("palsgd_outer_kernel", "outer", cfg, peak, peak_src, outer_ms, outer_bytes, n_outer,
                                 units_per_launch=Pn, launches_inside_step_loop=in_loop_outer,
                                 launches_timed_alone=n_outer - in_loop_outer,
                                 note="launches inside the step loop plus launches timed on their own right "
                                      "after it, each behind slots that inner steps have let diverge")
        cycle = None
        if r_inner["avg_ms"] and r_outer["avg_ms"]:
            # average cost per step of a whole synchronisation cycle: H inner launches + one outer sync
            cyc_ms = (cfg.H * r_inner["avg_ms"] + r_outer["avg_ms"]) / cfg.H
            cycle = {"H": cfg.H, "ms_per_step": cyc_ms, "value": K * Pn / (cyc_ms * 1e-3), "unit": UNIT,
                     "outer_share": r_outer["avg_ms"] / (cfg.H * cyc_ms),
                     "note": "(H * inner avg + outer avg) / H from the per-kernel CUDA-event times above"}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_total / args.steps,
            "higher_is_better": True, "scaling": "strong" if args.shard else "weak", "vs_baseline": None,
            "dtype": dtype_of(cfg),
            "data": "synthetic", "config": dict(workload_config(cfg, args), **layout_info),
            "roofline": r_inner,
            "roofline_outer": r_outer,
            "cycle": cycle,
            "roofline_ddp": (roofline_entry("palsgd_ddp_kernel", "ddp", cfg, peak, peak_src, ddp["ms"], ddp["bytes"],
                                            ddp["launches"], units_per_launch=Pn,
                                            note="timed outside the step loop; not part of value") if ddp else None),
            "ragged_layout": ({"layout": ragged["layout"], "n_segments": ragged["n_segments"],
                               "n_chunks": ragged["n_chunks"],
                               "roofline": roofline_entry("palsgd_inner_kernel", "inner", cfg, peak, peak_src,
                                                          ragged["inner_ms"], ragged["inner_bytes"], ragged["n_inner"],
                                                          traffic=None),
                               "roofline_outer": roofline_entry("palsgd_outer_kernel", "outer", cfg, peak, peak_src,
                                                                ragged["outer_ms"], ragged["outer_bytes"],
                                                                ragged["n_outer"], units_per_launch=Pn, traffic=None),
                               "note": "the same kernels over one allocation per (buffer kind, worker, tensor); "
                                       "timed on their own after the main regions; not part of value"}
                              if ragged else None),
            "outer_split": ({"partial": roofline_entry("palsgd_outer_partial_kernel", "outer", cfg, peak, peak_src,
                                                       split["partial_ms"], split["partial_bytes"], split["n"],
                                                       traffic=None),
                             "finish": roofline_entry("palsgd_outer_kernel (sum from the exchange buffer)", "outer", cfg,
                                                      peak, peak_src, split["finish_ms"], split["finish_bytes"],
                                                      split["n"], traffic=None),
                             "ddp_partial": roofline_entry("palsgd_ddp_partial_kernel", "ddp", cfg, peak, peak_src,
                                                           split["ddp_partial_ms"], split["ddp_partial_bytes"],
                                                           split["n"], traffic=None),
                             "ddp_finish": roofline_entry("palsgd_ddp_kernel (gradient sum from the exchange buffer)",
                                                          "ddp", cfg, peak, peak_src, split["ddp_finish_ms"],
                                                          split["ddp_finish_bytes"], split["n"], traffic=None),
                             "note": "outer sync and DDP warm-up step as local sum -> (all-reduce) -> finish, the form "
                                     "for workers spread over several GPUs; one GPU here, no collective; not part of "
                                     "value"}
                            if split else None),
            "graph_cycle": graph_cycle,
            "cpu_baseline": cpu_baseline,
            "e2e": ({"value": K * P_job * e2e["steps"] / (e2e["ms"] * 1e-3), "unit": UNIT,
                     "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                     "steps": e2e["steps"], "outer_syncs": e2e["syncs"]} if e2e else None),
            "gpu_launches": launches,
            "clocks": clocks,
        }
        print(json.dumps(line), flush=True)
    ctx.destroy()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(W.CONFIGS))
    ap.add_argument("--e2e-steps", type=int, default=0, help="0 = min(steps, H)")
    ap.add_argument("--inner-variant", type=int, default=0, help="palsgd_set_tuning(INNER_VARIANT); 0 = default")
    ap.add_argument("--grad-clip", type=float, default=0.0,
                    help="global-norm clip threshold (adds the norm pass to every step); 0 = off, the benchmark default")
    ap.add_argument("--shard", action="store_true",
                    help="N > 1: one model sharded over the ranks along the parameter axis (strong scaling, no "
                         "exchange) instead of one replica of the workload per rank")
    ap.add_argument("--workers", action="store_true",
                    help="spread the K workers over the ranks (K / N each) and run the outer sync around an NCCL "
                         "all-reduce: the paper's own deployment; not the default")
    ap.add_argument("--layout", choices=["arena", "separate", "misaligned"], default="arena",
                    help="device layout of the tensor list: packed (K, P) arenas (default), one allocation per "
                         "(worker, tensor, buffer kind), or packed and shifted off 16-byte alignment")
    ap.add_argument("--outer-launches", type=int, default=8,
                    help="outer-sync launches timed on their own after the step loop")
    ap.add_argument("--no-outer", action="store_true", help="skip the separate timing of the outer-sync kernel")
    ap.add_argument("--no-ragged", action="store_true",
                    help="skip the separate timing of the inner and outer kernels on the one-allocation-per-tensor layout")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="skip the separate timing of the graph-captured cycle")
    ap.add_argument("--no-ddp", action="store_true", help="skip the separate timing of the DDP warm-up kernel")
    args = ap.parse_args()
    cfg = W.get_config(args.workload)
    if args.impl == "reference":
        if args.steps == 256:
            args.steps = 32                       # a bounded sample: keep the CPU run to about a minute
        run_reference(args, cfg)
    elif args.workers:
        run_workers(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
