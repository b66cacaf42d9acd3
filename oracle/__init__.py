"""PALSGD CPU oracle (ctypes front end).   TEST INFRASTRUCTURE ONLY.

A plain, slow statement of Algorithm 1 and of the optimizers it names, in C
(`palsgd_oracle_impl.c`, `palsgd_oracle_common.c`), loaded here through ctypes.
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; it shares no code with the CUDA library and neither imports the
other.

Parity status: every function below is pinned by `tests/test_oracle_*.py`
(library routines of torch.optim / cuRAND's host generator, closed forms, exact
rational brute force, a hand trace, invariants).  Nothing here is "parity
unpinned".
"""
from __future__ import annotations

import ctypes as C
from typing import Optional

import numpy as np

from . import build as _build

_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        path = _build.build()
        L = C.CDLL(str(path))
        L.palsgd_oracle_philox4x32_10.argtypes = [C.POINTER(C.c_uint32)] * 3
        L.palsgd_oracle_philox4x32_10.restype = None
        L.palsgd_oracle_threshold.argtypes = [C.c_double]
        L.palsgd_oracle_threshold.restype = C.c_uint64
        L.palsgd_oracle_draw_word.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32]
        L.palsgd_oracle_draw_word.restype = C.c_uint32
        L.palsgd_oracle_decision.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_double]
        L.palsgd_oracle_decision.restype = C.c_int
        L.palsgd_oracle_bf16_to_f32.argtypes = [C.c_uint16]
        L.palsgd_oracle_bf16_to_f32.restype = C.c_float
        L.palsgd_oracle_bf16_from_f32.argtypes = [C.c_float]
        L.palsgd_oracle_bf16_from_f32.restype = C.c_uint16
        L.palsgd_oracle_bf16_from_f64.argtypes = [C.c_double]
        L.palsgd_oracle_bf16_from_f64.restype = C.c_uint16
        for name, ct in (("f32", C.c_float), ("f64", C.c_double), ("bf16", C.c_uint16)):
            f = getattr(L, f"palsgd_oracle_sumsq_{name}")
            f.argtypes = [C.POINTER(ct), C.c_uint64]
            f.restype = C.c_double
        L.palsgd_oracle_clip_coef.argtypes = [C.c_double, C.c_double]
        L.palsgd_oracle_clip_coef.restype = C.c_double
        L.palsgd_oracle_schedule.argtypes = [C.c_int, C.c_uint64, C.c_uint64, C.c_uint64, C.c_double,
                                             C.c_double, C.c_double]
        L.palsgd_oracle_schedule.restype = C.c_double
        L.palsgd_oracle_set_threads.argtypes = [C.c_int]
        L.palsgd_oracle_set_threads.restype = None
        L.palsgd_oracle_get_threads.argtypes = []
        L.palsgd_oracle_get_threads.restype = C.c_int
        _lib = L
    return _lib


def philox4x32_10(ctr, key) -> np.ndarray:
    c = (C.c_uint32 * 4)(*[int(v) & 0xFFFFFFFF for v in ctr])
    k = (C.c_uint32 * 2)(*[int(v) & 0xFFFFFFFF for v in key])
    o = (C.c_uint32 * 4)()
    lib().palsgd_oracle_philox4x32_10(c, k, o)
    return np.array(list(o), dtype=np.uint32)


def threshold(p: float) -> int:
    return int(lib().palsgd_oracle_threshold(float(p)))


def draw_word(seed: int, t: int, k: int) -> int:
    return int(lib().palsgd_oracle_draw_word(int(seed), int(t), int(k)))


def decision(seed: int, t: int, k: int, p: float) -> int:
    return int(lib().palsgd_oracle_decision(int(seed), int(t), int(k), float(p)))


def bf16_from_f32(f: float) -> int:
    return int(lib().palsgd_oracle_bf16_from_f32(float(np.float32(f))))


def bf16_from_f64(d: float) -> int:
    return int(lib().palsgd_oracle_bf16_from_f64(float(d)))


def bf16_to_f32(h: int) -> float:
    return float(lib().palsgd_oracle_bf16_to_f32(int(h)))


def sumsq(g: np.ndarray) -> float:
    """Exact sum of squares of a float32 / float64 array, or of bf16 bit patterns (uint16),
    rounded once to binary64."""
    g = np.ascontiguousarray(g).reshape(-1)
    name, ct = {np.dtype(np.float32): ("f32", C.c_float), np.dtype(np.float64): ("f64", C.c_double),
                np.dtype(np.uint16): ("bf16", C.c_uint16)}[g.dtype]
    return float(getattr(lib(), f"palsgd_oracle_sumsq_{name}")(g.ctypes.data_as(C.POINTER(ct)), g.size))


def clip_coef(sumsq_: float, max_norm: float) -> float:
    return float(lib().palsgd_oracle_clip_coef(float(sumsq_), float(max_norm)))


def schedule(kind: int, t: int, warmup: int, total: int, base: float, min_value: float = 0.0,
             start_factor: float = 0.0) -> float:
    """Linear warm-up, then constant (kind 0) or cosine annealing (kind 1)."""
    return float(lib().palsgd_oracle_schedule(int(kind), int(t), int(warmup), int(total), float(base),
                                              float(min_value), float(start_factor)))


def set_threads(n: int) -> None:
    lib().palsgd_oracle_set_threads(int(n))


def get_threads() -> int:
    return int(lib().palsgd_oracle_get_threads())


def _state_struct(real):
    ptr = C.POINTER(real)

    class State(C.Structure):
        _fields_ = [
            ("K", C.c_uint32), ("H", C.c_uint64), ("p", C.c_double), ("inner", C.c_int32),
            ("beta1", C.c_double), ("beta2", C.c_double), ("eps", C.c_double),
            ("weight_decay", C.c_double), ("momentum", C.c_double),
            ("outer_lr", C.c_double), ("outer_momentum", C.c_double),
            ("outer_nesterov", C.c_int32), ("seed", C.c_uint64), ("precision", C.c_int32),
            ("P", C.c_uint64),
            ("x", ptr), ("m", ptr), ("v", ptr), ("xg", ptr), ("u", ptr),
            ("xw", C.POINTER(C.c_uint16)),
            ("t", C.c_uint64), ("s", C.POINTER(C.c_uint64)), ("n_outer", C.c_uint64),
            ("pow1", C.POINTER(C.c_double)), ("pow2", C.POINTER(C.c_double)),
            ("last_b", C.POINTER(C.c_uint8)),
            ("max_grad_norm", C.c_double), ("forced_sumsq", C.POINTER(C.c_double)),
            ("sumsq", C.POINTER(C.c_double)), ("clipc", C.POINTER(C.c_double)),
            ("outer_opt", C.c_int32), ("outer_beta1", C.c_double), ("outer_beta2", C.c_double),
            ("outer_eps", C.c_double), ("outer_weight_decay", C.c_double), ("uv", ptr),
            ("opow1", C.c_double), ("opow2", C.c_double), ("sum_groups", C.c_uint32),
        ]

    return State


_STATE = {"f32": _state_struct(C.c_float), "f64": _state_struct(C.c_double)}
_NP = {"f32": np.float32, "f64": np.float64}
_CT = {"f32": C.c_float, "f64": C.c_double}


class Oracle:
    """K workers' state and the steps of Algorithm 1 over a flat model of P
    elements.  `x0` is (K, P) float32: the initial local models (mode 0) or
    initial masters (mode 1).  `dtype` picks the arithmetic: "f32" (parity
    reference) or "f64" (yard-stick)."""

    def __init__(self, x0: np.ndarray, *, K: int, H: int, p: float, inner: int = 0,
                 beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
                 weight_decay: float = 0.01, momentum: float = 0.0,
                 outer_lr: float = 0.7, outer_momentum: float = 0.9,
                 outer_nesterov: bool = True, seed: int = 0, precision: int = 0,
                 max_grad_norm: float = 0.0, outer_opt: int = 0, outer_beta1: float = 0.9,
                 outer_beta2: float = 0.999, outer_eps: float = 1e-8, outer_weight_decay: float = 0.0,
                 sum_groups: int = 0, dtype: str = "f32"):
        x0 = np.asarray(x0)
        assert x0.ndim == 2 and x0.shape[0] == K, x0.shape
        self.dtype = dtype
        self.K, self.P = int(K), int(x0.shape[1])
        np_t, ct = _NP[dtype], _CT[dtype]
        self.x = np.ascontiguousarray(x0, dtype=np_t).copy()
        self.m = np.zeros_like(self.x)
        self.v = np.zeros_like(self.x)
        self.xg = np.zeros(self.P, dtype=np_t)
        self.u = np.zeros(self.P, dtype=np_t)
        self.uv = np.zeros(self.P, dtype=np_t) if outer_opt == 1 else None
        self.xw = np.zeros((self.K, self.P), dtype=np.uint16) if precision == 1 else None
        self.s = np.zeros(self.K, dtype=np.uint64)
        self.pow1 = np.ones(self.K, dtype=np.float64)
        self.pow2 = np.ones(self.K, dtype=np.float64)
        self.last_b = np.zeros(self.K, dtype=np.uint8)
        self.sumsq = np.zeros(self.K, dtype=np.float64)
        self.clipc = np.ones(self.K, dtype=np.float64)
        self._forced_sumsq = None
        S = _STATE[dtype]
        p_ = lambda a, t: a.ctypes.data_as(C.POINTER(t))
        self._st = S(
            K=K, H=H, p=p, inner=inner, beta1=beta1, beta2=beta2, eps=eps,
            weight_decay=weight_decay, momentum=momentum, outer_lr=outer_lr,
            outer_momentum=outer_momentum, outer_nesterov=int(bool(outer_nesterov)),
            seed=seed, precision=precision, P=self.P,
            x=p_(self.x, ct), m=p_(self.m, ct), v=p_(self.v, ct), xg=p_(self.xg, ct),
            u=p_(self.u, ct),
            xw=p_(self.xw, C.c_uint16) if self.xw is not None else None,
            t=0, s=p_(self.s, C.c_uint64), n_outer=0,
            pow1=p_(self.pow1, C.c_double), pow2=p_(self.pow2, C.c_double),
            last_b=p_(self.last_b, C.c_uint8),
            max_grad_norm=float(max_grad_norm), forced_sumsq=None,
            sumsq=p_(self.sumsq, C.c_double), clipc=p_(self.clipc, C.c_double),
            outer_opt=int(outer_opt), outer_beta1=outer_beta1, outer_beta2=outer_beta2,
            outer_eps=outer_eps, outer_weight_decay=outer_weight_decay,
            uv=p_(self.uv, ct) if self.uv is not None else None, opow1=1.0, opow2=1.0, sum_groups=0)
        self.K = int(K)
        self.set_sum_groups(sum_groups)          # before the initial global model is formed
        L = lib()
        sfx = dtype
        self._init = getattr(L, f"palsgd_oracle_init_{sfx}")
        self._inner = getattr(L, f"palsgd_oracle_inner_step_{sfx}")
        self._pull = getattr(L, f"palsgd_oracle_pseudo_sync_{sfx}")
        self._outer = getattr(L, f"palsgd_oracle_outer_sync_{sfx}")
        self._step = getattr(L, f"palsgd_oracle_step_{sfx}")
        self._ddp = getattr(L, f"palsgd_oracle_ddp_step_{sfx}")
        SP = C.POINTER(S)
        self._init.argtypes = [SP]; self._init.restype = None
        for f in (self._inner, self._step):
            f.argtypes = [SP, C.c_void_p, C.c_double, C.c_double, C.c_void_p]
            f.restype = C.c_int
        self._pull.argtypes = [SP, C.c_uint64, C.c_double]; self._pull.restype = None
        self._ddp.argtypes = [SP, C.c_void_p, C.c_double]; self._ddp.restype = None
        self._outer.argtypes = [SP]; self._outer.restype = None
        self.precision = precision
        self._init(C.byref(self._st))

    # counters ------------------------------------------------------------
    @property
    def t(self) -> int:
        return int(self._st.t)

    @property
    def n_outer(self) -> int:
        return int(self._st.n_outer)

    # workers spread over several machines ----------------------------------
    def set_sum_groups(self, groups: int) -> None:
        """Form the sum over the K workers (initial global model, outer sync) in two levels: `groups`
        machines of K/groups consecutive workers each add up their own workers first (ascending), then
        the partial sums are added in ascending order of the machines.  0 or 1: one level, ascending k.
        The constructor's `sum_groups` applies it to the initial global model as well."""
        groups = int(groups)
        if groups > 1 and self.K % groups != 0:
            raise ValueError("the workers do not divide evenly over the groups")
        self._st.sum_groups = groups

    # schedules -----------------------------------------------------------
    def set_outer_lr(self, lr: float) -> None:
        """The outer learning rate may follow a schedule (warm-up, then cosine annealing): it is
        an input of each synchronisation."""
        self._st.outer_lr = float(lr)

    # gradient clipping ---------------------------------------------------
    def set_grad_clip(self, max_norm: float) -> None:
        self._st.max_grad_norm = float(max_norm)

    def force_sumsq(self, sumsq_per_worker) -> None:
        """Use these K sums of squares in the following steps instead of computing them from the
        gradients passed in (for replays of a sample of a large run); None switches back."""
        if sumsq_per_worker is None:
            self._forced_sumsq = None
            self._st.forced_sumsq = None
        else:
            self._forced_sumsq = np.ascontiguousarray(sumsq_per_worker, dtype=np.float64)
            assert self._forced_sumsq.shape == (self.K,)
            self._st.forced_sumsq = self._forced_sumsq.ctypes.data_as(C.POINTER(C.c_double))

    # steps ---------------------------------------------------------------
    def _grads_ptr(self, grads: np.ndarray):
        want = np.float32 if self.precision == 0 else np.uint16
        g = np.ascontiguousarray(grads, dtype=want)
        assert g.shape == (self.K, self.P), (g.shape, (self.K, self.P))
        return g, g.ctypes.data_as(C.c_void_p)

    @staticmethod
    def _forced_ptr(forced):
        if forced is None:
            return None, None
        f = np.ascontiguousarray(forced, dtype=np.uint8)
        return f, f.ctypes.data_as(C.c_void_p)

    def inner_step(self, grads, lr_t: float, eta_t: float, forced=None) -> None:
        g, gp = self._grads_ptr(grads)
        f, fp = self._forced_ptr(forced)
        rc = self._inner(C.byref(self._st), gp, float(lr_t), float(eta_t), fp)
        if rc:
            raise ValueError("undefined coefficient: pull with p=0 or gradient step with p=1")

    def step(self, grads, lr_t: float, eta_t: float, forced=None) -> None:
        g, gp = self._grads_ptr(grads)
        f, fp = self._forced_ptr(forced)
        rc = self._step(C.byref(self._st), gp, float(lr_t), float(eta_t), fp)
        if rc:
            raise ValueError("undefined coefficient: pull with p=0 or gradient step with p=1")

    def ddp_step(self, grads, lr_t: float) -> None:
        """One step of the DDP warm-up phase: averaged gradient, one InnerOPT step for all workers."""
        g, gp = self._grads_ptr(grads)
        self._ddp(C.byref(self._st), gp, float(lr_t))

    def pseudo_sync(self, worker_mask: int, beta: float) -> None:
        self._pull(C.byref(self._st), int(worker_mask), float(beta))

    def outer_sync(self) -> None:
        self._outer(C.byref(self._st))
