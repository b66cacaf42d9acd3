"""Test harness: runs the CUDA library and the CPU oracle on the same seeded
inputs and compares them.  Holds no arithmetic of the method itself."""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

import oracle
import paper_2504_18454_b200 as P

GUARD = 64                  # sentinel elements on both sides of every arena row
SENTINEL = 1536.0            # exactly representable in bf16 too
REL_TOL, ABS_FLOOR = 1e-6, 1e-7   # fp32 state: max |rel err| <= 1e-6 with abs floor 1e-7


def cfg_kwargs(cfg) -> dict:
    return dict(K=cfg.K, H=cfg.H, p=cfg.p, inner=cfg.inner, beta1=cfg.beta1, beta2=cfg.beta2,
                eps=cfg.eps, weight_decay=cfg.weight_decay, momentum=cfg.momentum,
                outer_lr=cfg.outer_lr, outer_momentum=cfg.outer_momentum,
                outer_nesterov=cfg.outer_nesterov, seed=cfg.decision_seed, precision=cfg.precision,
                outer_opt=cfg.outer_opt, outer_beta1=cfg.outer_beta1, outer_beta2=cfg.outer_beta2,
                outer_eps=cfg.outer_eps, outer_weight_decay=cfg.outer_weight_decay)


def make_oracle(cfg, x0: np.ndarray, dtype: str = "f32") -> oracle.Oracle:
    return oracle.Oracle(x0, dtype=dtype, **cfg_kwargs(cfg))


class GpuRun:
    """The library over torch-owned buffers.

    layout: "arena"      one row per worker, tensors packed back to back (fused into one segment)
            "misaligned" as arena, shifted by one element (scalar path)
            "separate"   one allocation per (worker, tensor)
    """

    def __init__(self, cfg, x0: np.ndarray, numel: Optional[Sequence[int]] = None,
                 layout: str = "arena", device: str = "cuda:0", row_align: int = 8, shift: int = 1):
        self.cfg, self.layout, self.dev = cfg, layout, torch.device(device)
        self.numel = [int(n) for n in (numel if numel is not None else [t.numel for t in cfg.tensors])]
        self.K, self.Ptot = cfg.K, int(sum(self.numel))
        assert x0.shape == (self.K, self.Ptot)
        self.bf = cfg.precision == 1
        self.adam = cfg.inner == 0
        pdt = torch.bfloat16 if self.bf else torch.float32
        self.off = GUARD + (shift if layout == "misaligned" else 0)   # "misaligned": every row starts `shift` elements late
        self.starts = np.concatenate([[0], np.cumsum(self.numel)]).astype(np.int64)
        kinds = {"param": (pdt, self.K), "grad": (pdt, self.K), "m": (torch.float32, self.K),
                 "global_": (torch.float32, 1), "outer_mom": (torch.float32, 1)}
        if self.adam:
            kinds["v"] = (torch.float32, self.K)
        if self.bf:
            kinds["master"] = (torch.float32, self.K)
        if cfg.outer_opt == 1:
            kinds["outer_v"] = (torch.float32, 1)
        self.arena: Dict[str, torch.Tensor] = {}
        self.views: Dict[str, List[List[torch.Tensor]]] = {}
        row = (self.off + self.Ptot + GUARD + 8 + row_align - 1) // row_align * row_align   # elements per arena row
        for name, (dt, rows) in kinds.items():
            if layout == "separate":
                self.views[name] = [[torch.full((n,), SENTINEL, dtype=dt, device=self.dev)
                                     for n in self.numel] for _ in range(rows)]
            else:
                a = torch.full((rows, row), SENTINEL, dtype=dt, device=self.dev)
                self.arena[name] = a
                self.views[name] = [[a[r, self.off + self.starts[j]: self.off + self.starts[j + 1]]
                                     for j in range(len(self.numel))] for r in range(rows)]
        self._write("master" if self.bf else "param", x0)
        v = self.views
        self.stream = torch.cuda.current_stream(self.dev).cuda_stream
        self.lib = P.Palsgd(numel=self.numel, params=v["param"], grads=v["grad"], m=v["m"],
                            v=v.get("v"), master=v.get("master"), global_=v["global_"][0],
                            outer_mom=v["outer_mom"][0], outer_v=v["outer_v"][0] if "outer_v" in v else None,
                            stream=self.stream, **cfg_kwargs(cfg))

    # ---- moving data
    def _write(self, name: str, host: np.ndarray) -> None:
        rows = len(self.views[name])
        host = host.reshape(rows, self.Ptot)
        dt = self.views[name][0][0].dtype if self.numel else torch.float32
        t = torch.from_numpy(np.ascontiguousarray(host))
        if dt == torch.bfloat16:
            t = t.view(torch.int16).view(torch.bfloat16) if t.dtype in (torch.int16, torch.uint16) else t
        if self.layout == "separate":
            for r in range(rows):
                for j in range(len(self.numel)):
                    self.views[name][r][j].copy_(t[r, self.starts[j]:self.starts[j + 1]])
        else:
            self.arena[name][:, self.off:self.off + self.Ptot].copy_(t)

    def _read(self, name: str) -> np.ndarray:
        if self.layout == "separate":
            rows = [torch.cat([x.reshape(-1) for x in r]) if r else torch.empty(0) for r in self.views[name]]
            t = torch.stack(rows)
        else:
            t = self.arena[name][:, self.off:self.off + self.Ptot]
        t = t.contiguous()
        if t.dtype == torch.bfloat16:
            return t.view(torch.int16).cpu().numpy().view(np.uint16)
        return t.cpu().numpy()

    def set_grads(self, g: np.ndarray) -> None:
        """g: (K, P) float32, or uint16 bf16 bit patterns in mixed-precision mode."""
        if self.bf:
            g = np.ascontiguousarray(g, dtype=np.uint16).view(np.int16)
        self._write("grad", g)

    def state(self) -> Dict[str, np.ndarray]:
        torch.cuda.synchronize(self.dev)
        out = {"x": self._read("master" if self.bf else "param"), "m": self._read("m"),
               "xg": self._read("global_")[0], "u": self._read("outer_mom")[0]}
        if self.adam:
            out["v"] = self._read("v")
        if self.bf:
            out["xw"] = self._read("param")
        if "outer_v" in self.views:
            out["uv"] = self._read("outer_v")[0]
        return out

    def guards_intact(self) -> bool:
        if self.layout == "separate":
            return True
        torch.cuda.synchronize(self.dev)
        for name, a in self.arena.items():
            lo = a[:, :self.off].float()
            hi = a[:, self.off + self.Ptot:].float()
            if not bool((lo == SENTINEL).all()) or not bool((hi == SENTINEL).all()):
                return False
        return True

    # ---- the calls under test
    def step(self, lr, eta):
        self.lib.step(lr, eta, self.stream)

    def inner_step(self, lr, eta):
        self.lib.inner_step(lr, eta, self.stream)

    def outer_sync(self):
        self.lib.outer_sync(self.stream)

    def ddp_step(self, lr):
        self.lib.ddp_step(lr, self.stream)

    def set_grad_clip(self, max_norm):
        self.lib.set_grad_clip(max_norm)

    def set_outer_lr(self, lr):
        self.lib.set_outer_lr(lr)

    def grad_norms(self):
        return self.lib.get_grad_norms(self.stream)

    def pseudo_sync(self, mask, beta):
        self.lib.pseudo_sync(mask, beta, self.stream)

    def counters(self):
        return self.lib.get_counters(self.stream)


def ulp_distance(a: np.ndarray, b: np.ndarray) -> int:
    """Largest distance in units in the last place between two float32 arrays."""
    if a.size == 0:
        return 0
    def key(x):
        i = np.ascontiguousarray(x, dtype=np.float32).view(np.int32).astype(np.int64)
        return np.where(i < 0, -(i & 0x7FFFFFFF), i)
    return int(np.abs(key(a) - key(b)).max())


def compare_state(gpu: Dict[str, np.ndarray], orc: oracle.Oracle, *, rel=REL_TOL, floor=ABS_FLOOR,
                  names=("x", "m", "v", "xg", "u", "uv"), exact: bool = False) -> Dict[str, float]:
    """Element-by-element comparison.  Returns the worst relative error and ulp
    distance per array; raises on a violation of the tolerance (or of bitwise
    equality when exact=True)."""
    report = {}
    for n in names:
        if n not in gpu:
            continue
        a = gpu[n]
        b = np.asarray(getattr(orc, n), dtype=np.float64).reshape(a.shape)
        err = np.abs(a.astype(np.float64) - b) / np.maximum(np.abs(b), floor / rel)
        worst = float(err.max()) if err.size else 0.0
        ulps = ulp_distance(a, b.astype(np.float32)) if orc.dtype == "f32" else -1
        report[n] = (worst, ulps)
        assert worst <= rel, f"{n}: max rel err {worst:.3e} > {rel:.1e} (ulp distance {ulps})"
        if exact:
            assert ulps == 0, f"{n}: not bit-identical to the fp32 oracle (ulp distance {ulps})"
    if "xw" in gpu and orc.xw is not None:
        ga = gpu["xw"].astype(np.int32)
        oa = np.asarray(orc.xw).reshape(gpu["xw"].shape).astype(np.int32)
        same_sign = (ga >> 15) == (oa >> 15)
        d = np.abs((ga & 0x7FFF) - (oa & 0x7FFF))
        zero = ((ga & 0x7FFF) == 0) & ((oa & 0x7FFF) == 0)
        ok = (same_sign & (d <= 1)) | zero
        report["xw"] = (float(d.max()) if d.size else 0.0, int(d.max()) if d.size else 0)
        assert ok.all(), "bf16 working params differ from RNE(master) by more than 1 bf16 ulp"
        if exact:
            assert np.array_equal(gpu["xw"], np.asarray(orc.xw).reshape(gpu["xw"].shape))
    return report
