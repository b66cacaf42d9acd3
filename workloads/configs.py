"""The benchmark/parity configurations: hyper-parameters and sizes only."""
from __future__ import annotations

from dataclasses import dataclass, replace
from itertools import product
from typing import Callable, Dict, Iterator, List

from .shapes import (
    TensorSpec,
    flat_shape,
    gptneo_8m_shape,
    gptneo_125m_shape,
    resnet50_shape,
)

ADAMW, SGDM = 0, 1
FP32, BF16_MASTER = 0, 1


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    shape: Callable[[], List[TensorSpec]]
    K: int                      # workers (replica slots)
    H: int                      # outer-sync interval
    p: float                    # pseudo-sync probability
    eta: float                  # mixing rate eta_t (constant over t here)
    lr: float                   # inner learning rate alpha_t (constant over t here)
    T: int                      # inner steps of the full run
    inner: int = ADAMW
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.01
    momentum: float = 0.0       # inner SGD momentum
    outer_lr: float = 0.7
    outer_momentum: float = 0.9
    outer_nesterov: bool = True
    outer_opt: int = 0          # 0 SGD with (Nesterov) momentum, 1 AdamW on the outer gradient
    outer_beta1: float = 0.9
    outer_beta2: float = 0.999
    outer_eps: float = 1e-8
    outer_weight_decay: float = 0.0
    precision: int = FP32
    init_std: float = 0.02
    grad_std: float = 0.01
    param_seed: int = 1234
    grad_seed: int = 5678
    decision_seed: int = 2025

    @property
    def tensors(self) -> List[TensorSpec]:
        return self.shape()

    @property
    def P(self) -> int:
        return sum(t.numel for t in self.tensors)

    def with_(self, **kw) -> "WorkloadConfig":
        return replace(self, **kw)


CONFIGS: Dict[str, WorkloadConfig] = {
    # K=4 flat 2^20, AdamW, p=.25, H=8, 16 steps
    "c0_flat_1m": WorkloadConfig(
        name="c0_flat_1m", shape=lambda: flat_shape(1 << 20),
        K=4, H=8, p=0.25, eta=16.0, lr=1e-3, T=16),
    # GPT-Neo-8M-shaped, K=8, AdamW, p=.1, H=64, 256 steps
    "c1_gptneo8m": WorkloadConfig(
        name="c1_gptneo8m", shape=gptneo_8m_shape,
        K=8, H=64, p=0.1, eta=16.0, lr=1e-3, T=256),
    # ResNet-50-shaped, K=8, momentum SGD, p=.2, H=32, 128 steps
    "c2_resnet50": WorkloadConfig(
        name="c2_resnet50", shape=resnet50_shape,
        K=8, H=32, p=0.2, eta=0.5, lr=0.1, T=128,
        inner=SGDM, momentum=0.9, weight_decay=1e-4, grad_std=1e-3),
    # GPT-Neo-125M-shaped, bf16 working + fp32 master, K=8, p=.1, H=128, 512 steps
    "c3_gptneo125m_bf16": WorkloadConfig(
        name="c3_gptneo125m_bf16", shape=gptneo_125m_shape,
        K=8, H=128, p=0.1, eta=16.0, lr=1e-3, T=512, precision=BF16_MASTER),
    # profiling-sized stand-ins (a few GB, larger than L2) for ncu captures of the same kernels
    "prof_flat16m_bf16": WorkloadConfig(
        name="prof_flat16m_bf16", shape=lambda: flat_shape(1 << 24),
        K=8, H=8, p=0.1, eta=16.0, lr=1e-3, T=16, precision=BF16_MASTER),
    "prof_flat16m_fp32": WorkloadConfig(
        name="prof_flat16m_fp32", shape=lambda: flat_shape(1 << 24),
        K=8, H=8, p=0.1, eta=16.0, lr=1e-3, T=16),
}


def get_config(name: str) -> WorkloadConfig:
    return CONFIGS[name]


def sweep_points(max_state_bytes: int | None = None) -> Iterator[WorkloadConfig]:
    """Bandwidth sweep on flat fp32 buffers: K x P x p x H grid."""
    for K, logP, p, H in product((4, 8, 16, 32), (20, 24, 26, 28),
                                 (0.0, 0.1, 0.5, 1.0), (16, 64, 256)):
        P = 1 << logP
        if max_state_bytes is not None and K * P * 16 + 8 * P > max_state_bytes:
            continue
        yield WorkloadConfig(
            name=f"c4_K{K}_P2e{logP}_p{p}_H{H}", shape=(lambda P=P: flat_shape(P)),
            K=K, H=H, p=p, eta=16.0, lr=1e-3, T=2 * H)
