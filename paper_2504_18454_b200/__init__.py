"""PALSGD update / synchronisation path for NVIDIA B200 (sm_100a).

`Palsgd` is a thin ctypes binding over the C ABI in `include/palsgd.h`
(`libpalsgd.so`, built in-tree by `paper_2504_18454_b200.build`).  Every step of
the path runs in the library's CUDA kernels; this package only marshals
arguments.  PyTorch supplies device memory and streams.
"""
from .binding import (  # noqa: F401
    Palsgd,
    PalsgdError,
    decision,
    plan_layout,
    schedule_value,
    OUTER_SGD,
    OUTER_ADAMW,
    SCHED_WARMUP_CONSTANT,
    SCHED_WARMUP_COSINE,
    outer_sync_noalloc,
    NOALLOC_SCRATCH_BYTES,
    lib,
    strerror,
    INNER_ADAMW,
    INNER_SGDM,
    PREC_FP32,
    PREC_BF16_MASTER,
    TUNE_INNER_GRID_CAP,
    TUNE_OUTER_GRID_CAP,
    TUNE_INNER_VARIANT,
    TUNE_OUTER_SUB_ELEMS,
    TUNE_DDP_SUB_ELEMS,
    TUNE_DDP_VARIANT,
    TUNE_OUTER_VARIANT,
    TUNE_OUTER_DYNAMIC,
)
