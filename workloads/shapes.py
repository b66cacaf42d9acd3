"""Parameter-list shapes of the models the paper trains (Appendix B, "Workloads").

Only element counts matter to the update/synchronisation path, so a model is a
list of (name, shape, init-kind) records.  The lists are produced from each
architecture's published construction rule, not from any model file.
"""
from __future__ import annotations

from dataclasses import dataclass
from math import prod
from typing import List, Tuple


@dataclass(frozen=True)
class TensorSpec:
    name: str
    shape: Tuple[int, ...]
    # how the synthetic initial value is drawn:
    #   "normal"  -> N(0, std^2)         (std given by the workload config)
    #   "kaiming" -> N(0, 2 / fan_in)    (fan_in = prod(shape[1:]))
    #   "ones" / "zeros" -> constant
    init: str = "normal"

    @property
    def numel(self) -> int:
        return int(prod(self.shape))

    @property
    def fan_in(self) -> int:
        return int(prod(self.shape[1:])) if len(self.shape) > 1 else int(self.shape[0])


def flat_shape(P: int) -> List[TensorSpec]:
    """One flat vector of P elements."""
    return [TensorSpec("flat", (int(P),), "normal")]


def _transformer_block(prefix: str, d: int, d_ff: int) -> List[TensorSpec]:
    return [
        TensorSpec(f"{prefix}.ln1.w", (d,)),
        TensorSpec(f"{prefix}.ln1.b", (d,)),
        TensorSpec(f"{prefix}.qkv.w", (d, 3 * d)),
        TensorSpec(f"{prefix}.qkv.b", (3 * d,)),
        TensorSpec(f"{prefix}.proj.w", (d, d)),
        TensorSpec(f"{prefix}.proj.b", (d,)),
        TensorSpec(f"{prefix}.ln2.w", (d,)),
        TensorSpec(f"{prefix}.ln2.b", (d,)),
        TensorSpec(f"{prefix}.fc.w", (d, d_ff)),
        TensorSpec(f"{prefix}.fc.b", (d_ff,)),
        TensorSpec(f"{prefix}.fc2.w", (d_ff, d)),
        TensorSpec(f"{prefix}.fc2.b", (d,)),
    ]


def gptneo_8m_shape() -> List[TensorSpec]:
    """GPT-Neo-8M-like list: vocabulary 8192, width 256, 8 blocks, MLP 1024.

    99 tensors, 8,415,744 elements.
    """
    d, d_ff, vocab, layers = 256, 1024, 8192, 8
    out = [TensorSpec("wte", (vocab, d))]
    for i in range(layers):
        out += _transformer_block(f"h{i}", d, d_ff)
    out += [TensorSpec("ln_f.w", (d,)), TensorSpec("ln_f.b", (d,))]
    return out


def gptneo_125m_shape() -> List[TensorSpec]:
    """GPT-Neo-125M-like list: vocabulary 50257, 2048 positions, width 768,
    12 blocks, MLP 3072.  148 tensors, 125,226,240 elements.
    """
    d, d_ff, vocab, n_pos, layers = 768, 3072, 50257, 2048, 12
    out = [TensorSpec("wte", (vocab, d)), TensorSpec("wpe", (n_pos, d))]
    for i in range(layers):
        out += _transformer_block(f"h{i}", d, d_ff)
    out += [TensorSpec("ln_f.w", (d,)), TensorSpec("ln_f.b", (d,))]
    return out


def resnet50_shape() -> List[TensorSpec]:
    """ResNet-50 list from the bottleneck construction rule: a 7x7 stem, four
    stages of [3, 4, 6, 3] bottleneck blocks with widths 64/128/256/512 and
    expansion 4, a 1x1 projection on the first block of each stage, and a
    1000-way classifier.  161 tensors, 25,557,032 elements.
    """
    out: List[TensorSpec] = []

    def conv(name, c_out, c_in, k):
        out.append(TensorSpec(name, (c_out, c_in, k, k), "kaiming"))

    def bn(name, c):
        out.append(TensorSpec(f"{name}.scale", (c,), "ones"))
        out.append(TensorSpec(f"{name}.bias", (c,), "zeros"))

    conv("stem.conv", 64, 3, 7)
    bn("stem.bn", 64)
    c_in = 64
    for s, (blocks, w) in enumerate(zip([3, 4, 6, 3], [64, 128, 256, 512])):
        for b in range(blocks):
            p = f"s{s}.b{b}"
            conv(f"{p}.conv1", w, c_in, 1)
            bn(f"{p}.bn1", w)
            conv(f"{p}.conv2", w, w, 3)
            bn(f"{p}.bn2", w)
            conv(f"{p}.conv3", 4 * w, w, 1)
            bn(f"{p}.bn3", 4 * w)
            if b == 0:
                conv(f"{p}.down.conv", 4 * w, c_in, 1)
                bn(f"{p}.down.bn", 4 * w)
            c_in = 4 * w
    out.append(TensorSpec("fc.w", (1000, 2048), "kaiming"))
    out.append(TensorSpec("fc.b", (1000,), "zeros"))
    return out
