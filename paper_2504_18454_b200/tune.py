"""Launch-shape sweep for the PALSGD kernels on the GPU at hand.

    python -m paper_2504_18454_b200.tune WORKLOAD [--variants 0,1,6,7] [--chunks 4096,8192]
                                                  [--outer-subs 1024,2048] [--steps 40]

For every chunk size (fixed at palsgd_init through PALSGD_CHUNK_ELEMS, hence one
child process each) it times the fused inner kernel for every compiled variant
and the outer kernel for every slice size, with CUDA events on the launching
stream, and prints achieved GB/s = algorithmic bytes / time.  Results never
depend on these knobs; only speed does.
"""
from __future__ import annotations

import argparse
import os
import time
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _inner_bytes(cfg, pull: bool) -> int:
    bf = cfg.precision == 1
    if pull:
        return 14 if bf else 12
    if cfg.inner == 0:
        return 28
    return 18 if bf else 20


def _child(args) -> None:
    import torch
    import workloads as W
    import paper_2504_18454_b200 as P
    from paper_2504_18454_b200.arena import ReplicaArena

    cfg = W.get_config(args.workload)
    dev = torch.device("cuda:0")
    numel = [t.numel for t in cfg.tensors]
    arena = ReplicaArena(numel, cfg.K, precision=cfg.precision, inner=cfg.inner, device=dev)
    arena.model.normal_(0, cfg.init_std)
    for k in range(cfg.K):
        arena.rows("grad")[k].copy_(torch.randn(cfg.P, device=dev).mul_(cfg.grad_std))
    stream = torch.cuda.current_stream().cuda_stream
    ctx = arena.make_context(stream=stream, H=cfg.H, p=cfg.p, beta1=cfg.beta1, beta2=cfg.beta2, eps=cfg.eps,
                             weight_decay=cfg.weight_decay, momentum=cfg.momentum, outer_lr=cfg.outer_lr,
                             outer_momentum=cfg.outer_momentum, outer_nesterov=cfg.outer_nesterov,
                             seed=cfg.decision_seed)
    chunk = os.environ.get("PALSGD_CHUNK_ELEMS", "default")

    def time_inner(steps, warm=4):
        ctx.set_counters(0, [0] * cfg.K, 0, stream)            # same decision sequence for every variant
        for _ in range(warm):
            ctx.inner_step(cfg.lr, cfg.eta, stream)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        ev[0].record()
        for i in range(steps):
            ctx.inner_step(cfg.lr, cfg.eta, stream)
            ev[i + 1].record()
        torch.cuda.synchronize()
        ms = sum(ev[i].elapsed_time(ev[i + 1]) for i in range(steps))
        byts = sum(_inner_bytes(cfg, bool(P.decision(cfg.decision_seed, warm + i, k, cfg.p)))
                   for i in range(steps) for k in range(cfg.K)) * cfg.P
        return byts / ms / 1e6

    def time_outer(reps=8):
        heat()
        for _ in range(2):
            ctx.outer_sync(stream)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            ctx.outer_sync(stream)
        e1.record()
        torch.cuda.synchronize()
        per = (10 if cfg.precision == 1 else 8) * cfg.K + 16
        return per * cfg.P / (e0.elapsed_time(e1) / reps) / 1e6

    def heat():
        # optional: load the GPU for a while first, so that the timing sees the clocks of a long run
        if args.heat_ms > 0:
            ctx.set_grad_clip(0.0)
            t0 = time.time()
            while (time.time() - t0) * 1e3 < args.heat_ms:
                for _ in range(16):
                    ctx.inner_step(cfg.lr, cfg.eta, stream)
                torch.cuda.synchronize()

    def time_ddp(reps=8):
        heat()
        for _ in range(2):
            ctx.ddp_step(cfg.lr, stream)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            ctx.ddp_step(cfg.lr, stream)
        e1.record()
        torch.cuda.synchronize()
        per = (16 if cfg.inner == 0 else 12) * (cfg.K + 1)      # both precisions: see include/palsgd.h
        return per * cfg.P / (e0.elapsed_time(e1) / reps) / 1e6

    def time_norm(steps, ddp=False, warm=3):
        # the norm pass alone = (clipped step) - (unclipped step), both timed over the same decisions
        def loop(n):
            ctx.set_counters(0, [0] * cfg.K, 0, stream)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for i in range(warm + n):
                if i == warm:
                    e0.record()
                ctx.ddp_step(cfg.lr, stream) if ddp else ctx.inner_step(cfg.lr, cfg.eta, stream)
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1)
        ctx.set_grad_clip(0.0); base = loop(steps)
        ctx.set_grad_clip(1.0); clipped = loop(steps)
        ctx.set_grad_clip(0.0)
        gsz = 2 if cfg.precision == 1 else 4
        if ddp:
            byts = steps * cfg.K * cfg.P * gsz
        else:
            byts = sum(0 if P.decision(cfg.decision_seed, warm + i, k, cfg.p) else gsz
                       for i in range(steps) for k in range(cfg.K)) * cfg.P
        return byts / (clipped - base) / 1e6, (clipped - base) / steps, base / steps

    def time_pull(reps=8):
        mask = (1 << cfg.K) - 1
        for _ in range(2):
            ctx.pseudo_sync(mask, 0.1, stream)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            ctx.pseudo_sync(mask, 0.1, stream)
        e1.record()
        torch.cuda.synchronize()
        per = 14 if cfg.precision == 1 else 12
        return per * cfg.K * cfg.P / (e0.elapsed_time(e1) / reps) / 1e6

    r = sorted(time_pull() for _ in range(3))
    print(f"{cfg.name} chunk={chunk} forced pull of all workers: {r[1]:.0f} GB/s (runs {r[0]:.0f}..{r[2]:.0f}; "
          f"x_g shared through L2, so the floor is below the 12/14 B per element assumed)", flush=True)
    for v in args.variants:
        ctx.set_tuning(P.TUNE_INNER_VARIANT, v)
        r = sorted(time_inner(args.steps) for _ in range(3))
        print(f"{cfg.name} chunk={chunk} inner variant={v}: {r[1]:.0f} GB/s (runs {r[0]:.0f}..{r[2]:.0f})", flush=True)
    for ddp in (False, True):
        r = sorted(time_norm(args.steps, ddp) for _ in range(3))[1]
        print(f"{cfg.name} chunk={chunk} grad-norm pass ({'ddp' if ddp else 'per worker'}): {r[0]:.0f} GB/s of gradient "
              f"bytes, {r[1]:.3f} ms on top of a {r[2]:.3f} ms step", flush=True)
    for sub, dyn in [(s_, d_) for s_ in args.outer_subs for d_ in args.outer_dynamic]:
        ctx.set_tuning(P.TUNE_OUTER_DYNAMIC, dyn)
        chunk = f"{os.environ.get('PALSGD_CHUNK_ELEMS', 'default')} dyn={dyn}"
        ctx.set_tuning(P.TUNE_OUTER_SUB_ELEMS, sub)
        for variant in (1, 2):
            ctx.set_tuning(P.TUNE_OUTER_VARIANT, variant)
            r = sorted(time_outer() for _ in range(3))
            print(f"{cfg.name} chunk={chunk} outer slice={sub} variant={variant}: {r[1]:.0f} GB/s "
                  f"(runs {r[0]:.0f}..{r[2]:.0f})", flush=True)
        ctx.set_tuning(P.TUNE_DDP_SUB_ELEMS, sub)
        for variant in (1, 2):
            ctx.set_tuning(P.TUNE_DDP_VARIANT, variant)
            r = sorted(time_ddp() for _ in range(3))
            print(f"{cfg.name} chunk={chunk} ddp slice={sub} variant={variant}: {r[1]:.0f} GB/s "
                  f"(runs {r[0]:.0f}..{r[2]:.0f})", flush=True)
    ctx.destroy()


def main() -> None:
    ints = lambda s: [int(x) for x in s.split(",") if x]
    ap = argparse.ArgumentParser(description=__doc__.splitlines()[0])
    ap.add_argument("workload")
    ap.add_argument("--variants", type=ints, default=[0])
    ap.add_argument("--chunks", type=ints, default=[])
    ap.add_argument("--outer-subs", type=ints, default=[1024])
    ap.add_argument("--outer-dynamic", type=ints, default=[0], help="CTAs per SM of the persistent outer/DDP grid; 0 = off")
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--heat-ms", type=float, default=0.0,
                    help="run inner steps for this long before each outer/DDP timing (power-capped clocks)")
    ap.add_argument("--child", action="store_true", help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.child or not args.chunks:
        _child(args)
        return
    for ce in args.chunks:
        env = dict(os.environ, PALSGD_CHUNK_ELEMS=str(ce))
        cmd = [sys.executable, "-m", "paper_2504_18454_b200.tune", args.workload, "--child",
               "--variants", ",".join(map(str, args.variants)),
               "--outer-subs", ",".join(map(str, args.outer_subs)), "--steps", str(args.steps),
               "--outer-dynamic", ",".join(map(str, args.outer_dynamic)), "--heat-ms", str(args.heat_ms)]
        subprocess.run(cmd, env=env, check=True, cwd=ROOT)


if __name__ == "__main__":
    main()
