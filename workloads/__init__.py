"""Synthetic workloads for the PALSGD update/synchronisation path.

This package holds parameter-list *shapes* and *seeded input generators* only.
It contains none of the method's arithmetic (no optimizer step, no pull, no
averaging, no decision draw): both the CPU oracle's tests and the CUDA path's
tests/benchmarks draw their inputs from here, and neither imports the other.
"""
from .shapes import (  # noqa: F401
    flat_shape,
    gptneo_8m_shape,
    gptneo_125m_shape,
    resnet50_shape,
    TensorSpec,
)
from .configs import CONFIGS, WorkloadConfig, get_config, sweep_points  # noqa: F401
from .generate import (  # noqa: F401
    init_params_host,
    grads_host,
    bf16_bits_from_f32_host,
    sample_indices,
)
