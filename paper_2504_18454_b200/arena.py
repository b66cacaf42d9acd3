"""Device-memory layout helper: K replica slots as rows of flat torch arenas.

Each buffer kind (params, grads, moments, master) is ONE (K, P) allocation whose
row k is worker k's tensor list packed back to back; the global model and the
outer momentum are (P,) vectors.  Packed tensors are adjacent in every buffer,
so the library fuses the whole list into a single segment and every chunk but
the last is full.  This module only allocates and slices: no arithmetic.
"""
from __future__ import annotations

from typing import Dict, List, Sequence

import torch

from .binding import INNER_ADAMW, PREC_BF16_MASTER, Palsgd


class ReplicaArena:
    def __init__(self, numel: Sequence[int], K: int, *, precision: int, inner: int,
                 device: torch.device | str = "cuda", outer_adamw: bool = False):
        self.numel = [int(n) for n in numel]
        self.K, self.P = int(K), int(sum(self.numel))
        self.precision, self.inner = precision, inner
        self.device = torch.device(device)
        bf = precision == PREC_BF16_MASTER
        pdt = torch.bfloat16 if bf else torch.float32
        Ppad = (self.P + 63) // 64 * 64          # rows stay 128-byte aligned
        mk = lambda rows, dt: torch.zeros((rows, Ppad), dtype=dt, device=self.device)
        self.t: Dict[str, torch.Tensor] = {
            "param": mk(K, pdt), "grad": mk(K, pdt), "m": mk(K, torch.float32),
            "global_": mk(1, torch.float32), "outer_mom": mk(1, torch.float32)}
        if inner == INNER_ADAMW:
            self.t["v"] = mk(K, torch.float32)
        if bf:
            self.t["master"] = mk(K, torch.float32)
        if outer_adamw:                          # second moment of AdamW as OuterOPT
            self.t["outer_v"] = mk(1, torch.float32)
        starts = [0]
        for n in self.numel:
            starts.append(starts[-1] + n)
        self.starts = starts

    def rows(self, name: str) -> torch.Tensor:
        """(K, P) (or (1, P)) view of a buffer kind without the row padding."""
        return self.t[name][:, :self.P]

    def views(self, name: str) -> List[List[torch.Tensor]]:
        a = self.t[name]
        return [[a[r, self.starts[j]:self.starts[j + 1]] for j in range(len(self.numel))]
                for r in range(a.shape[0])]

    @property
    def model(self) -> torch.Tensor:
        """The fp32 local models: params (fp32 mode) or masters (mixed precision)."""
        return self.rows("master" if self.precision == PREC_BF16_MASTER else "param")

    def bytes_allocated(self) -> int:
        return sum(a.numel() * a.element_size() for a in self.t.values())

    def make_context(self, *, stream: int, **cfg) -> Palsgd:
        v = {k: self.views(k) for k in self.t}
        return Palsgd(K=self.K, numel=self.numel, params=v["param"], grads=v["grad"], m=v["m"],
                      v=v.get("v"), master=v.get("master"), global_=v["global_"][0],
                      outer_mom=v["outer_mom"][0], outer_v=v["outer_v"][0] if "outer_v" in v else None,
                      precision=self.precision, inner=self.inner, stream=stream, **cfg)
