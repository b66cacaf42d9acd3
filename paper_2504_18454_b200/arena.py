"""Device-memory layout helper: K replica slots over torch-owned buffers.

Three layouts of the same tensor list:

  "arena"       each buffer kind (params, grads, moments, master) is ONE (K, P)
                allocation whose row k is worker k's tensor list packed back to
                back; the global model and the outer momentum are (P,) vectors.
                Packed tensors are adjacent in every buffer, so the library fuses
                the whole list into a single segment.
  "separate"    one allocation per (buffer kind, worker, tensor), the way a
                framework holds its parameters; every allocation carries a gap
                behind it, so no two tensors are adjacent and the library keeps
                one segment per tensor (a ragged list: a partial chunk at the end
                of every tensor, tensors far smaller than a chunk).
  "misaligned"  as "arena", shifted by one element, so that no buffer is 16-byte
                aligned: the library peels a scalar head off the front and runs
                the rest on its vector path.

This module only allocates, slices and copies: no arithmetic.
"""
from __future__ import annotations

from typing import Dict, List, Sequence

import torch

from .binding import INNER_ADAMW, PREC_BF16_MASTER, Palsgd

LAYOUTS = ("arena", "separate", "misaligned")
_GAP = 128                  # elements between separately allocated tensors' ends and the next block


class ReplicaArena:
    def __init__(self, numel: Sequence[int], K: int, *, precision: int, inner: int,
                 device: torch.device | str = "cuda", outer_adamw: bool = False, layout: str = "arena"):
        if layout not in LAYOUTS:
            raise ValueError(f"layout must be one of {LAYOUTS}")
        self.numel = [int(n) for n in numel]
        self.K, self.P = int(K), int(sum(self.numel))
        self.precision, self.inner, self.layout = precision, inner, layout
        self.device = torch.device(device)
        bf = precision == PREC_BF16_MASTER
        pdt = torch.bfloat16 if bf else torch.float32
        kinds = {"param": (K, pdt), "grad": (K, pdt), "m": (K, torch.float32),
                 "global_": (1, torch.float32), "outer_mom": (1, torch.float32)}
        if inner == INNER_ADAMW:
            kinds["v"] = (K, torch.float32)
        if bf:
            kinds["master"] = (K, torch.float32)
        if outer_adamw:                          # second moment of AdamW as OuterOPT
            kinds["outer_v"] = (1, torch.float32)
        starts = [0]
        for n in self.numel:
            starts.append(starts[-1] + n)
        self.starts = starts
        self.t: Dict[str, torch.Tensor] = {}                 # packed layouts: one tensor per kind
        self._views: Dict[str, List[List[torch.Tensor]]] = {}
        self._shift = 1 if layout == "misaligned" else 0
        if layout == "separate":
            self._blocks = []                                # keeps the padded allocations alive
            for name, (rows, dt) in kinds.items():
                per_row = []
                for _ in range(rows):
                    row = []
                    for n in self.numel:
                        blk = torch.zeros(n + _GAP, dtype=dt, device=self.device)
                        self._blocks.append(blk)
                        row.append(blk[:n])
                    per_row.append(row)
                self._views[name] = per_row
        else:
            Ppad = (self.P + self._shift + 255) // 256 * 256  # rows start on multiples of 256 elements (1024 bytes of fp32)
            for name, (rows, dt) in kinds.items():
                a = torch.zeros((rows, Ppad), dtype=dt, device=self.device)
                self.t[name] = a
                s = self._shift
                self._views[name] = [[a[r, s + starts[j]: s + starts[j + 1]] for j in range(len(self.numel))]
                                     for r in range(rows)]

    # ---- access
    def rows(self, name: str) -> torch.Tensor:
        """(K, P) (or (1, P)) view of a buffer kind (packed layouts only)."""
        if self.layout == "separate":
            raise ValueError("rows() needs a packed layout; use write_flat / read_flat")
        return self.t[name][:, self._shift:self._shift + self.P]

    def views(self, name: str) -> List[List[torch.Tensor]]:
        return self._views[name]

    def has(self, name: str) -> bool:
        return name in self._views

    @property
    def model_name(self) -> str:
        """The buffer kind holding the fp32 local models: params (fp32 mode) or masters (mixed precision)."""
        return "master" if self.precision == PREC_BF16_MASTER else "param"

    @property
    def model(self) -> torch.Tensor:
        return self.rows(self.model_name)

    def write_flat(self, name: str, row: int, flat: torch.Tensor) -> None:
        """Copy a (P,) tensor (the tensor list concatenated) into row `row` of buffer kind `name`."""
        if self.layout == "separate":
            for j, v in enumerate(self._views[name][row]):
                v.copy_(flat[self.starts[j]:self.starts[j + 1]])
        else:
            self.rows(name)[row].copy_(flat)

    def read_flat(self, name: str, row: int) -> torch.Tensor:
        """Row `row` of buffer kind `name` as one (P,) tensor (a copy for the separate layout)."""
        if self.layout == "separate":
            return torch.cat([v.reshape(-1) for v in self._views[name][row]])
        return self.rows(name)[row]

    def bytes_allocated(self) -> int:
        if self.layout == "separate":
            return sum(b.numel() * b.element_size() for b in self._blocks)
        return sum(a.numel() * a.element_size() for a in self.t.values())

    def make_context(self, *, stream: int, **cfg) -> Palsgd:
        v = self._views
        return Palsgd(K=self.K, numel=self.numel, params=v["param"], grads=v["grad"], m=v["m"],
                      v=v.get("v"), master=v.get("master"), global_=v["global_"][0],
                      outer_mom=v["outer_mom"][0], outer_v=v["outer_v"][0] if "outer_v" in v else None,
                      precision=self.precision, inner=self.inner, stream=stream, **cfg)
