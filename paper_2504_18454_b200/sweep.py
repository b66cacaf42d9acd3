"""Bandwidth sweep of the PALSGD kernels on flat fp32 buffers.

    python -m paper_2504_18454_b200.sweep [--K 4,8,16,32] [--logP 20,24,26,28] [--p 0,0.1,0.5,1]
                                          [--H 16,64,256] [--steps 24] [--peak-gbs X]

For every (K, P) the K replica slots are allocated once; the fused inner kernel
is timed for every pseudo-sync probability p (its time does not depend on H) and
the outer-sync kernel once.  Achieved GB/s = algorithmic bytes / CUDA-event time,
where the inner bytes follow the decisions actually drawn in the timed steps
(28 B per worker-element on a gradient step, 12 B on a pull; AdamW, fp32) and the
outer bytes are (8K + 16) per parameter.  The average cost per step of a whole
H-step cycle, (H * inner + outer) / H, is derived for every H.  A point is run when its
state plus a 4 GB margin fits in the device memory that is free once the previous point's
buffers have been released; otherwise the row says what was free.  Output: a Markdown table.
"""
from __future__ import annotations

import argparse
import gc
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main() -> None:
    import torch
    import paper_2504_18454_b200 as P
    from paper_2504_18454_b200.arena import ReplicaArena

    floats = lambda s: [float(x) for x in s.split(",") if x]
    ints = lambda s: [int(x) for x in s.split(",") if x]
    ap = argparse.ArgumentParser(description=__doc__.splitlines()[0])
    ap.add_argument("--K", type=ints, default=[4, 8, 16, 32])
    ap.add_argument("--logP", type=ints, default=[20, 24, 26, 28])
    ap.add_argument("--p", type=floats, default=[0.0, 0.1, 0.5, 1.0])
    ap.add_argument("--H", type=ints, default=[16, 64, 256])
    ap.add_argument("--steps", type=int, default=24)
    ap.add_argument("--peak-gbs", type=float, default=0.0, help="0 = MEASURED_PEAKS.json, else 6650")
    ap.add_argument("--outer-sub", type=int, default=0, help="palsgd_set_tuning(OUTER_SUB_ELEMS); 0 = default")
    args = ap.parse_args()

    peak = args.peak_gbs
    if peak <= 0:
        try:
            peak = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["hbm_gbs"])
        except Exception:
            peak = 6650.0
    dev = torch.device("cuda:0")
    stream = torch.cuda.current_stream(dev).cuda_stream
    seed, lr, eta = 2025, 1e-3, 16.0

    print(f"peak = {peak:.1f} GB/s; {args.steps} timed inner launches per point after 4 warm-up launches; "
          f"8 timed outer launches; AdamW inner, Nesterov outer (0.7 / 0.9), eta = {eta}")
    hdr = ["K", "P", "state GB", "p", "pulls", "inner ms", "inner GB/s", "frac", "worker-elem upd/s",
           "outer ms", "outer GB/s", "frac"] + [f"ms/step H={h}" for h in args.H]
    print("| " + " | ".join(hdr) + " |")
    print("|" + "---|" * len(hdr))
    for K in args.K:
        for logP in args.logP:
            Pn = 1 << logP
            need = K * Pn * 16 + 8 * Pn
            gc.collect()
            torch.cuda.empty_cache()
            free, _ = torch.cuda.mem_get_info(dev)
            if need + (4 << 30) > free:
                print(f"| {K} | 2^{logP} | {need / 1e9:.1f} | skipped: state + 4 GB margin exceeds the {free / 1e9:.0f} GB free |")
                continue
            arena = ReplicaArena([Pn], K, precision=P.PREC_FP32, inner=P.INNER_ADAMW, device=dev)
            arena.model.normal_(0, 0.02)
            for k in range(K):
                arena.rows("grad")[k].normal_(0, 0.01)
            outer = None
            for p in args.p:
                ctx = arena.make_context(stream=stream, H=1 << 30, p=p, seed=seed)
                for _ in range(4):
                    ctx.inner_step(lr, eta, stream)
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
                ev[0].record()
                for _ in range(args.steps):
                    ctx.inner_step(lr, eta, stream)
                ev[1].record()
                torch.cuda.synchronize(dev)
                ms = ev[0].elapsed_time(ev[1]) / args.steps
                pulls = sum(P.decision(seed, 4 + i, k, p) for i in range(args.steps) for k in range(K))
                byts = (28 * (K * args.steps - pulls) + 12 * pulls) * Pn / args.steps
                if outer is None:
                    if args.outer_sub:
                        ctx.set_tuning(P.TUNE_OUTER_SUB_ELEMS, args.outer_sub)
                    for _ in range(2):
                        ctx.outer_sync(stream)
                    ev[0].record()
                    for _ in range(8):
                        ctx.outer_sync(stream)
                    ev[1].record()
                    torch.cuda.synchronize(dev)
                    oms = ev[0].elapsed_time(ev[1]) / 8
                    outer = (oms, (8 * K + 16) * Pn / oms / 1e6)
                gbs = byts / ms / 1e6
                row = [K, f"2^{logP}", f"{need / 1e9:.2f}", p, f"{pulls}/{K * args.steps}", f"{ms:.4f}",
                       f"{gbs:.0f}", f"{gbs / peak:.3f}", f"{K * Pn / ms * 1e3:.3e}",
                       f"{outer[0]:.4f}", f"{outer[1]:.0f}", f"{outer[1] / peak:.3f}"]
                row += [f"{(h * ms + outer[0]) / h:.4f}" for h in args.H]
                print("| " + " | ".join(map(str, row)) + " |", flush=True)
                ctx.destroy()
                del ctx                                  # the context keeps its tensors alive
            del arena


if __name__ == "__main__":
    main()
