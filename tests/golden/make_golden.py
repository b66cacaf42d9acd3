"""Writes tests/golden/oracle_tiny_run.txt by calling only `oracle/` (and the
seeded input generators).  The file freezes the oracle's own output on a tiny
run, so that any later change to its arithmetic shows up as a diff that has to
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


if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_tiny_run.txt")
    with open(out, "w") as f:
        f.write(render())
    print("wrote", out)
