"""Writes tests/golden/oracle_tiny_run.txt and oracle_widened_run.txt by calling only
`oracle/` (and the seeded input generators).  The files freeze the oracle's own output on tiny
runs, so that any later change to its arithmetic shows up as a diff that has to
be justified against the paper.  Run:  python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from workloads import flat_shape, grads_host, init_params_host  # noqa: E402

CASES = {
    # name: (inner, precision)
    "adamw_fp32": (0, 0),
    "sgdm_fp32": (1, 0),
    "adamw_bf16": (0, 1),
}
K, P, H, T, p, eta, lr, seed = 4, 24, 4, 10, 0.25, 16.0, 1e-3, 2025


def run(inner, precision):
    from workloads import bf16_bits_from_f32_host
    x0 = np.tile(init_params_host(flat_shape(P), 1234, 0.02), (K, 1))
    o = oracle.Oracle(x0, dtype="f32", K=K, H=H, p=p, inner=inner, momentum=0.9 if inner else 0.0,
                      seed=seed, precision=precision)
    bits = []
    for t in range(T):
        g = np.stack([grads_host(P, 5678, t, k, 0.01) for k in range(K)])
        o.step(bf16_bits_from_f32_host(g) if precision else g, lr, eta)
        bits.append("".join(str(int(b)) for b in o.last_b))
    return o, bits


def render():
    lines = ["# oracle (f32 instantiation) on K=4 P=24 H=4 T=10 p=0.25 eta=16 lr=1e-3 seed=2025",
             "# written by tests/golden/make_golden.py; values are binary32 bit patterns"]
    for name, (inner, precision) in CASES.items():
        o, bits = run(inner, precision)
        lines.append(f"[{name}]")
        lines.append("decisions " + " ".join(bits))
        lines.append("s " + " ".join(str(int(v)) for v in o.s))
        lines.append(f"t {o.t} n_outer {o.n_outer}")
        lines.append("xg " + " ".join(f"{v:08x}" for v in o.xg.view(np.uint32)))
        lines.append("x3 " + " ".join(f"{v:08x}" for v in o.x[3].view(np.uint32)))
        lines.append("u " + " ".join(f"{v:08x}" for v in o.u.view(np.uint32)))
        if precision:
            lines.append("xw3 " + " ".join(f"{v:04x}" for v in o.xw[3]))
    return "\n".join(lines) + "\n"


def render_widened():
    """A second tiny run over the later additions: 3 DDP warm-up steps, then Algorithm 1 with
    global-norm clipping and AdamW as OuterOPT under a scheduled outer learning rate."""
    from workloads import bf16_bits_from_f32_host
    lines = ["# oracle (f32 instantiation): 3 DDP steps + 9 steps of Algorithm 1, K=4 P=24 H=3 p=0.25 eta=16 lr=1e-3,",
             "# clip 0.03, AdamW outer (lr schedule: warm-up 1 + cosine to 4 rounds, base 0.02, floor 0.002, start 0.5)",
             "# written by tests/golden/make_golden.py; binary32 / binary64 bit patterns"]
    for name, precision in (("widened_fp32", 0), ("widened_bf16", 1)):
        x0 = np.tile(init_params_host(flat_shape(P), 1234, 0.02), (K, 1))
        o = oracle.Oracle(x0, dtype="f32", K=K, H=3, p=p, inner=0, seed=seed, precision=precision,
                          max_grad_norm=0.03, outer_opt=1, outer_lr=0.02, outer_beta2=0.95, outer_weight_decay=0.05)
        sums = []
        for t in range(12):
            g = np.stack([grads_host(P, 5678, t, k, 0.01) for k in range(K)])
            g = bf16_bits_from_f32_host(g) if precision else g
            if t < 3:
                o.ddp_step(g, lr)
            else:
                o.set_outer_lr(oracle.schedule(1, o.n_outer, 1, 4, 0.02, 0.002, 0.5))
                o.step(g, lr, eta)
            sums.append(" ".join(f"{v:016x}" for v in o.sumsq.view(np.uint64)))
        lines.append(f"[{name}]")
        lines.append("s " + " ".join(str(int(v)) for v in o.s) + f" t {o.t} n_outer {o.n_outer}")
        lines.append("sumsq_last " + sums[-1])
        lines.append("sumsq_ddp " + sums[2])
        lines.append("clip " + " ".join(f"{v:016x}" for v in o.clipc.view(np.uint64)))
        lines.append("xg " + " ".join(f"{v:08x}" for v in o.xg.view(np.uint32)))
        lines.append("x2 " + " ".join(f"{v:08x}" for v in o.x[2].view(np.uint32)))
        lines.append("u " + " ".join(f"{v:08x}" for v in o.u.view(np.uint32)))
        lines.append("uv " + " ".join(f"{v:08x}" for v in o.uv.view(np.uint32)))
    return "\n".join(lines) + "\n"


if __name__ == "__main__":
    here = os.path.dirname(os.path.abspath(__file__))
    for fname, text in (("oracle_tiny_run.txt", render()), ("oracle_widened_run.txt", render_widened())):
        with open(os.path.join(here, fname), "w") as f:
            f.write(text)
        print("wrote", os.path.join(here, fname))
