"""ctypes binding of include/palsgd.h: same names, argument marshalling only."""
from __future__ import annotations

import ctypes as C
from pathlib import Path
from typing import List, Optional, Sequence

HERE = Path(__file__).resolve().parent
LIB_PATH = HERE / "libpalsgd.so"

INNER_ADAMW, INNER_SGDM = 0, 1
PREC_FP32, PREC_BF16_MASTER = 0, 1
OUTER_SGD, OUTER_ADAMW = 0, 1
SCHED_WARMUP_CONSTANT, SCHED_WARMUP_COSINE = 0, 1
TUNE_INNER_GRID_CAP, TUNE_OUTER_GRID_CAP, TUNE_INNER_VARIANT = 0, 1, 2
TUNE_OUTER_SUB_ELEMS, TUNE_DDP_SUB_ELEMS, TUNE_DDP_VARIANT = 5, 6, 7
TUNE_OUTER_VARIANT, TUNE_OUTER_DYNAMIC = 8, 9
MAX_WORKERS = 64


class PalsgdError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: {strerror(status)} ({status})" + (f": {detail}" if detail else ""))


class Config(C.Structure):
    _fields_ = [
        ("K", C.c_uint32), ("inner", C.c_int32), ("H", C.c_uint64), ("p", C.c_double),
        ("beta1", C.c_double), ("beta2", C.c_double), ("eps", C.c_double),
        ("weight_decay", C.c_double), ("momentum", C.c_double),
        ("outer_lr", C.c_double), ("outer_momentum", C.c_double),
        ("outer_nesterov", C.c_int32), ("precision", C.c_int32), ("seed", C.c_uint64),
        ("outer_opt", C.c_int32), ("reserved_", C.c_int32),
        ("outer_beta1", C.c_double), ("outer_beta2", C.c_double), ("outer_eps", C.c_double),
        ("outer_weight_decay", C.c_double),
    ]


class Buffers(C.Structure):
    _fields_ = [(n, C.POINTER(C.c_void_p)) for n in
                ("param", "grad", "master", "m", "v", "global_", "outer_mom", "outer_v")]


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """Load libpalsgd.so.  There is no fallback: a missing library is an error."""
    global _lib
    if _lib is not None:
        return _lib
    if not LIB_PATH.exists():
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2504_18454_b200.build` "
            "(needs nvcc); this package has no CPU or PyTorch fallback")
    L = C.CDLL(str(LIB_PATH))
    vp, u64p, u8p = C.c_void_p, C.POINTER(C.c_uint64), C.POINTER(C.c_uint8)
    L.palsgd_init.argtypes = [C.POINTER(vp), C.POINTER(Config), C.c_size_t, u64p, C.POINTER(Buffers), vp]
    L.palsgd_inner_step.argtypes = [vp, C.c_double, C.c_double, vp]
    L.palsgd_pseudo_sync.argtypes = [vp, C.c_uint64, C.c_double, vp]
    L.palsgd_cycle_capture.argtypes = [vp, C.c_double, C.c_double]
    L.palsgd_cycle_capture.restype = C.c_int
    L.palsgd_cycle_launch.argtypes = [vp, vp]
    L.palsgd_cycle_launch.restype = C.c_int
    L.palsgd_ddp_step.argtypes = [vp, C.c_double, vp]
    L.palsgd_ddp_step.restype = C.c_int
    L.palsgd_set_outer_lr.argtypes = [vp, C.c_double]
    L.palsgd_set_outer_lr.restype = C.c_int
    L.palsgd_schedule_value.argtypes = [C.c_int, C.c_uint64, C.c_uint64, C.c_uint64, C.c_double, C.c_double,
                                        C.c_double]
    L.palsgd_schedule_value.restype = C.c_double
    L.palsgd_set_grad_clip.argtypes = [vp, C.c_double]
    L.palsgd_set_grad_clip.restype = C.c_int
    L.palsgd_get_grad_norms.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_float), vp]
    L.palsgd_get_grad_norms.restype = C.c_int
    L.palsgd_outer_sync.argtypes = [vp, vp]
    L.palsgd_step.argtypes = [vp, C.c_double, C.c_double, vp]
    L.palsgd_step_host.argtypes = [vp, C.POINTER(vp), C.c_double, C.c_double, C.POINTER(vp), u8p,
                                   C.POINTER(C.c_int), vp]
    L.palsgd_get_counters.argtypes = [vp, u64p, u64p, u64p, u8p, vp]
    L.palsgd_set_counters.argtypes = [vp, C.c_uint64, u64p, C.c_uint64, vp]
    L.palsgd_get_launch_count.argtypes = [vp, u64p]
    L.palsgd_set_tuning.argtypes = [vp, C.c_int, C.c_int64]
    L.palsgd_exchange_numel.argtypes = [vp, u64p]
    L.palsgd_set_worker_offset.argtypes = [vp, C.c_uint32]
    L.palsgd_outer_partial.argtypes = [vp, vp, vp]
    L.palsgd_outer_finish.argtypes = [vp, vp, C.c_uint32, vp]
    L.palsgd_global_from_exchange.argtypes = [vp, vp, C.c_uint32, vp]
    L.palsgd_plan_layout.argtypes = [C.POINTER(Config), C.c_size_t, u64p, C.POINTER(Buffers), u64p, u64p,
                                     C.POINTER(C.c_uint32), u64p, u64p, C.POINTER(C.c_int32)]
    L.palsgd_plan_layout.restype = C.c_int
    L.palsgd_ddp_partial.argtypes = [vp, vp, vp]
    L.palsgd_ddp_finish.argtypes = [vp, vp, C.c_uint32, C.c_double, vp]
    for name in ("palsgd_exchange_numel", "palsgd_set_worker_offset", "palsgd_outer_partial", "palsgd_outer_finish",
                 "palsgd_global_from_exchange", "palsgd_ddp_partial", "palsgd_ddp_finish"):
        getattr(L, name).restype = C.c_int
    L.palsgd_get_layout.argtypes = [vp, u64p, u64p, C.POINTER(C.c_uint32)]
    L.palsgd_get_layout.restype = C.c_int
    L.palsgd_decision.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_double]
    for name in ("palsgd_init", "palsgd_inner_step", "palsgd_pseudo_sync", "palsgd_outer_sync",
                 "palsgd_step", "palsgd_step_host", "palsgd_get_counters", "palsgd_set_counters",
                 "palsgd_get_launch_count", "palsgd_set_tuning", "palsgd_decision"):
        getattr(L, name).restype = C.c_int
    L.palsgd_outer_sync_noalloc.argtypes = [C.c_uint32, C.c_int32, C.c_size_t, u64p, C.POINTER(vp), C.POINTER(vp),
                                            C.POINTER(vp), C.POINTER(vp), C.c_double, C.c_double, C.c_int32, vp]
    L.palsgd_outer_sync_noalloc.restype = C.c_int
    L.palsgd_strerror.argtypes = [C.c_int]
    L.palsgd_strerror.restype = C.c_char_p
    L.palsgd_last_cuda_error.argtypes = [vp]
    L.palsgd_last_cuda_error.restype = C.c_char_p
    L.palsgd_destroy.argtypes = [vp]
    L.palsgd_destroy.restype = None
    _lib = L
    return L


def strerror(status: int) -> str:
    return lib().palsgd_strerror(int(status)).decode()


def decision(seed: int, t: int, k: int, p: float) -> int:
    """palsgd_decision: the branch draw of Algorithm 1 as a pure host function."""
    rc = lib().palsgd_decision(int(seed), int(t), int(k), float(p))
    if rc < 0:
        raise PalsgdError(rc, "palsgd_decision")
    return rc


def schedule_value(kind: int, t: int, warmup: int, total: int, base: float, min_value: float = 0.0,
                   start_factor: float = 0.0) -> float:
    """palsgd_schedule_value: linear warm-up, then constant or cosine annealing (pure host function)."""
    return float(lib().palsgd_schedule_value(int(kind), int(t), int(warmup), int(total), float(base),
                                             float(min_value), float(start_factor)))


def _ptr_array(ptrs: Sequence[int]):
    return (C.c_void_p * len(ptrs))(*[C.c_void_p(int(p)) for p in ptrs])


def _data_ptrs(per_worker: Sequence[Sequence]) -> List[int]:
    """[k][j] tensors (anything with .data_ptr()) -> flat [k*n + j] addresses."""
    return [int(t.data_ptr()) for row in per_worker for t in row]


NOALLOC_SCRATCH_BYTES = 1 << 20


def outer_sync_noalloc(*, K: int, numel: Sequence[int], params, global_, outer_mom, master=None,
                       outer_lr: float = 0.7, outer_momentum: float = 0.9, outer_nesterov: bool = True,
                       precision: int = PREC_FP32, stream: int = 0) -> None:
    """palsgd_outer_sync_noalloc: the outer synchronisation for callers that may not allocate
    device memory (no context; the launch tables go into a fixed array inside the library).
    params/master: K lists of n tensors; global_/outer_mom: n tensors.  Calls whose GPU work
    could overlap race on that array: keep them on one stream."""
    n = len(numel)
    nm = (C.c_uint64 * n)(*[int(x) for x in numel])
    cast = lambda a: C.cast(a, C.POINTER(C.c_void_p))
    rc = lib().palsgd_outer_sync_noalloc(
        int(K), int(precision), n, nm, cast(_ptr_array(_data_ptrs(params))),
        cast(_ptr_array(_data_ptrs(master))) if master is not None else None,
        cast(_ptr_array([int(t.data_ptr()) for t in global_])),
        cast(_ptr_array([int(t.data_ptr()) for t in outer_mom])),
        float(outer_lr), float(outer_momentum), int(bool(outer_nesterov)), C.c_void_p(stream))
    if rc:
        raise PalsgdError(rc, "palsgd_outer_sync_noalloc")


def plan_layout(*, K: int, numel: Sequence[int], param, grad, m, global_, outer_mom, v=None, master=None,
                outer_v=None, inner: int = INNER_ADAMW, precision: int = PREC_FP32, outer_opt: int = OUTER_SGD):
    """What palsgd_init would make of a tensor list, from ADDRESSES alone (plain integers; nothing is
    dereferenced and no GPU is needed): param / grad / m / v / master are K rows of len(numel) addresses,
    global_ / outer_mom / outer_v one row.  Returns the segment and chunk counts and, per segment,
    (first tensor, tensors fused, scalar head)."""
    n = len(numel)
    cfg = Config(K=K, inner=inner, H=1, p=0.5, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, momentum=0.0,
                 outer_lr=1.0, outer_momentum=0.0, outer_nesterov=0, precision=precision, seed=0,
                 outer_opt=outer_opt, reserved_=0, outer_beta1=0.9, outer_beta2=0.999, outer_eps=1e-8,
                 outer_weight_decay=0.0)
    flat = lambda rows: _ptr_array([int(a) for row in rows for a in row])
    arrs = {"param": flat(param), "grad": flat(grad), "m": flat(m),
            "master": flat(master) if master is not None else None, "v": flat(v) if v is not None else None,
            "global_": _ptr_array([int(a) for a in global_]), "outer_mom": _ptr_array([int(a) for a in outer_mom]),
            "outer_v": _ptr_array([int(a) for a in outer_v]) if outer_v is not None else None}
    bufs = Buffers(**{k: (C.cast(a, C.POINTER(C.c_void_p)) if a is not None else None) for k, a in arrs.items()})
    nm = (C.c_uint64 * n)(*[int(x) for x in numel])
    ns, nc, ce = C.c_uint64(0), C.c_uint64(0), C.c_uint32(0)
    first, count, head = (C.c_uint64 * n)(), (C.c_uint64 * n)(), (C.c_int32 * n)()
    rc = lib().palsgd_plan_layout(C.byref(cfg), n, nm, C.byref(bufs), C.byref(ns), C.byref(nc), C.byref(ce),
                                  first, count, head)
    if rc:
        raise PalsgdError(rc, "palsgd_plan_layout")
    return {"n_segments": ns.value, "n_chunks": nc.value, "chunk_elems": ce.value,
            "segments": [(first[i], count[i], head[i]) for i in range(ns.value)]}


class Palsgd:
    """One PALSGD context over caller-owned device tensors.

    params/grads/m/v/master: K lists of n tensors (worker-major); global_/outer_mom:
    n tensors.  The tensors must stay alive as long as this object.  `stream`
    arguments are raw cudaStream_t values (e.g. torch.cuda.current_stream().cuda_stream).
    """

    def __init__(self, *, K: int, H: int, p: float, numel: Sequence[int],
                 params, grads, m, v=None, master=None, global_, outer_mom,
                 inner: int = INNER_ADAMW, beta1: float = 0.9, beta2: float = 0.999,
                 eps: float = 1e-8, weight_decay: float = 0.01, momentum: float = 0.0,
                 outer_lr: float = 0.7, outer_momentum: float = 0.9, outer_nesterov: bool = True,
                 precision: int = PREC_FP32, seed: int = 0, stream: int = 0,
                 outer_opt: int = OUTER_SGD, outer_v=None, outer_beta1: float = 0.9, outer_beta2: float = 0.999,
                 outer_eps: float = 1e-8, outer_weight_decay: float = 0.0):
        self._ctx = C.c_void_p()
        self.K, self.H, self.n = int(K), int(H), len(numel)
        self.numel = [int(x) for x in numel]
        self._keep = (params, grads, m, v, master, global_, outer_mom, outer_v)
        cfg = Config(K=K, inner=inner, H=H, p=p, beta1=beta1, beta2=beta2, eps=eps,
                     weight_decay=weight_decay, momentum=momentum, outer_lr=outer_lr,
                     outer_momentum=outer_momentum, outer_nesterov=int(bool(outer_nesterov)),
                     precision=precision, seed=seed, outer_opt=outer_opt, reserved_=0,
                     outer_beta1=outer_beta1, outer_beta2=outer_beta2, outer_eps=outer_eps,
                     outer_weight_decay=outer_weight_decay)
        arrs = {
            "param": _ptr_array(_data_ptrs(params)),
            "grad": _ptr_array(_data_ptrs(grads)),
            "master": _ptr_array(_data_ptrs(master)) if master is not None else None,
            "m": _ptr_array(_data_ptrs(m)),
            "v": _ptr_array(_data_ptrs(v)) if v is not None else None,
            "global_": _ptr_array([int(t.data_ptr()) for t in global_]),
            "outer_mom": _ptr_array([int(t.data_ptr()) for t in outer_mom]),
            "outer_v": _ptr_array([int(t.data_ptr()) for t in outer_v]) if outer_v is not None else None,
        }
        bufs = Buffers(**{k: (C.cast(a, C.POINTER(C.c_void_p)) if a is not None else None)
                          for k, a in arrs.items()})
        nm = (C.c_uint64 * self.n)(*self.numel)
        rc = lib().palsgd_init(C.byref(self._ctx), C.byref(cfg), self.n, nm, C.byref(bufs),
                               C.c_void_p(stream))
        if rc:
            detail = lib().palsgd_last_cuda_error(None).decode() if rc == -3 else ""
            self._ctx = C.c_void_p()
            raise PalsgdError(rc, "palsgd_init", detail)

    # -- helpers
    def _check(self, rc: int, where: str) -> None:
        if rc:
            detail = lib().palsgd_last_cuda_error(self._ctx).decode() if rc == -3 else ""
            raise PalsgdError(rc, where, detail)

    # -- the C ABI, one method per entry point
    def inner_step(self, lr_t: float, eta_t: float, stream: int = 0) -> None:
        self._check(lib().palsgd_inner_step(self._ctx, lr_t, eta_t, C.c_void_p(stream)), "palsgd_inner_step")

    def ddp_step(self, lr_t: float, stream: int = 0) -> None:
        self._check(lib().palsgd_ddp_step(self._ctx, lr_t, C.c_void_p(stream)), "palsgd_ddp_step")

    def pseudo_sync(self, worker_mask: int, beta: float, stream: int = 0) -> None:
        self._check(lib().palsgd_pseudo_sync(self._ctx, worker_mask, beta, C.c_void_p(stream)), "palsgd_pseudo_sync")

    def outer_sync(self, stream: int = 0) -> None:
        self._check(lib().palsgd_outer_sync(self._ctx, C.c_void_p(stream)), "palsgd_outer_sync")

    def step(self, lr_t: float, eta_t: float, stream: int = 0) -> None:
        self._check(lib().palsgd_step(self._ctx, lr_t, eta_t, C.c_void_p(stream)), "palsgd_step")

    def cycle_capture(self, lr_t: float, eta_t: float) -> None:
        self._check(lib().palsgd_cycle_capture(self._ctx, lr_t, eta_t), "palsgd_cycle_capture")

    def cycle_launch(self, stream: int = 0) -> None:
        self._check(lib().palsgd_cycle_launch(self._ctx, C.c_void_p(stream)), "palsgd_cycle_launch")

    def step_host(self, h_grad_ptrs, lr_t: float, eta_t: float, h_global_ptrs=None,
                  h_decisions_ptr: int = 0, stream: int = 0) -> bool:
        """h_grad_ptrs: ctypes array of K*n host addresses (see make_ptr_array);
        returns True when the step ended with an outer sync."""
        synced = C.c_int(0)
        rc = lib().palsgd_step_host(
            self._ctx, h_grad_ptrs, lr_t, eta_t, h_global_ptrs,
            C.cast(C.c_void_p(h_decisions_ptr), C.POINTER(C.c_uint8)) if h_decisions_ptr else None,
            C.byref(synced), C.c_void_p(stream))
        self._check(rc, "palsgd_step_host")
        return bool(synced.value)

    @staticmethod
    def make_ptr_array(ptrs: Sequence[int]):
        return _ptr_array(ptrs)

    def get_counters(self, stream: int = 0):
        t, n_outer = C.c_uint64(0), C.c_uint64(0)
        s = (C.c_uint64 * self.K)()
        b = (C.c_uint8 * self.K)()
        rc = lib().palsgd_get_counters(self._ctx, C.byref(t), s, C.byref(n_outer), b, C.c_void_p(stream))
        self._check(rc, "palsgd_get_counters")
        return {"t": t.value, "s": list(s), "n_outer": n_outer.value, "last_b": list(b)}

    def set_counters(self, t: int, s: Sequence[int], n_outer: int, stream: int = 0) -> None:
        arr = (C.c_uint64 * self.K)(*[int(x) for x in s])
        self._check(lib().palsgd_set_counters(self._ctx, t, arr, n_outer, C.c_void_p(stream)), "palsgd_set_counters")

    def set_outer_lr(self, outer_lr: float) -> None:
        self._check(lib().palsgd_set_outer_lr(self._ctx, outer_lr), "palsgd_set_outer_lr")

    def set_grad_clip(self, max_norm: float) -> None:
        self._check(lib().palsgd_set_grad_clip(self._ctx, max_norm), "palsgd_set_grad_clip")

    def get_grad_norms(self, stream: int = 0):
        ss, cl = (C.c_double * self.K)(), (C.c_float * self.K)()
        self._check(lib().palsgd_get_grad_norms(self._ctx, ss, cl, C.c_void_p(stream)), "palsgd_get_grad_norms")
        return list(ss), list(cl)

    def get_launch_count(self) -> int:
        n = C.c_uint64(0)
        self._check(lib().palsgd_get_launch_count(self._ctx, C.byref(n)), "palsgd_get_launch_count")
        return n.value

    def exchange_numel(self) -> int:
        n = C.c_uint64(0)
        self._check(lib().palsgd_exchange_numel(self._ctx, C.byref(n)), "palsgd_exchange_numel")
        return n.value

    def set_worker_offset(self, k0: int) -> None:
        self._check(lib().palsgd_set_worker_offset(self._ctx, int(k0)), "palsgd_set_worker_offset")

    def outer_partial(self, exchange_ptr: int, stream: int = 0) -> None:
        self._check(lib().palsgd_outer_partial(self._ctx, C.c_void_p(exchange_ptr), C.c_void_p(stream)),
                    "palsgd_outer_partial")

    def outer_finish(self, exchange_ptr: int, K_total: int, stream: int = 0) -> None:
        self._check(lib().palsgd_outer_finish(self._ctx, C.c_void_p(exchange_ptr), int(K_total), C.c_void_p(stream)),
                    "palsgd_outer_finish")

    def ddp_partial(self, exchange_ptr: int, stream: int = 0) -> None:
        self._check(lib().palsgd_ddp_partial(self._ctx, C.c_void_p(exchange_ptr), C.c_void_p(stream)), "palsgd_ddp_partial")

    def ddp_finish(self, exchange_ptr: int, K_total: int, lr_t: float, stream: int = 0) -> None:
        self._check(lib().palsgd_ddp_finish(self._ctx, C.c_void_p(exchange_ptr), int(K_total), lr_t, C.c_void_p(stream)),
                    "palsgd_ddp_finish")

    def global_from_exchange(self, exchange_ptr: int, K_total: int, stream: int = 0) -> None:
        self._check(lib().palsgd_global_from_exchange(self._ctx, C.c_void_p(exchange_ptr), int(K_total),
                                                      C.c_void_p(stream)), "palsgd_global_from_exchange")

    def get_layout(self):
        ns, nc, ce = C.c_uint64(0), C.c_uint64(0), C.c_uint32(0)
        self._check(lib().palsgd_get_layout(self._ctx, C.byref(ns), C.byref(nc), C.byref(ce)), "palsgd_get_layout")
        return {"n_segments": ns.value, "n_chunks": nc.value, "chunk_elems": ce.value}

    def set_tuning(self, knob: int, value: int) -> None:
        self._check(lib().palsgd_set_tuning(self._ctx, knob, value), "palsgd_set_tuning")

    def destroy(self) -> None:
        if self._ctx:
            lib().palsgd_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
