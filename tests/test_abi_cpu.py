"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every function include/palsgd.h declares, rejects bad arguments before any CUDA
call, and its host-side branch draw agrees with the oracle's."""
import ctypes as C
import os
import re

import pytest

import oracle
import paper_2504_18454_b200 as P
from paper_2504_18454_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "palsgd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(palsgd_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_entry_point():
    L = P.lib()
    names = _declared_functions()
    assert {"palsgd_init", "palsgd_inner_step", "palsgd_pseudo_sync", "palsgd_outer_sync",
            "palsgd_step", "palsgd_step_host", "palsgd_get_counters", "palsgd_set_counters",
            "palsgd_decision", "palsgd_strerror", "palsgd_destroy"} <= set(names)
    for n in names:
        assert hasattr(L, n), n


def test_config_struct_layout_matches_header():
    # K, inner, H, eight doubles (p .. outer_momentum), two int32, seed, two int32, four doubles: no padding
    assert C.sizeof(B.Config) == 4 + 4 + 8 + 8 * 8 + 4 + 4 + 8 + 4 + 4 + 4 * 8 == 136
    assert B.Config.H.offset == 8 and B.Config.seed.offset == 88 and B.Config.outer_beta1.offset == 104


def test_host_decision_matches_oracle_bit_for_bit():
    for seed in (0, 2025, 2**63 + 12345):
        for p in (0.0, 0.05, 0.1, 0.25, 0.5, 1.0):
            for t in list(range(64)) + [2**32 - 1, 2**32, 2**40 + 7]:
                for k in (0, 1, 7, 31, 63):
                    assert P.decision(seed, t, k, p) == oracle.decision(seed, t, k, p)


def test_decision_rejects_bad_arguments():
    for bad_p in (-0.1, 1.5, float("nan")):
        with pytest.raises(P.PalsgdError):
            P.decision(1, 0, 0, bad_p)
    # the worker index is the worker's index in the whole job: it may exceed one context's 64 slots
    assert P.decision(1, 0, 64, 0.5) == oracle.decision(1, 0, 64, 0.5)
    assert P.decision(9, 7, 1000, 0.5) == oracle.decision(9, 7, 1000, 0.5)


def test_strerror_covers_all_statuses():
    texts = {P.strerror(s) for s in (0, -1, -2, -3, -4, -5, -6, -8)}
    assert len(texts) == 8 and "unknown status" not in texts
    assert P.strerror(-99) == "unknown status" and P.strerror(-7) == "unknown status"


def _fake_init(**over):
    """palsgd_init with plausible non-NULL fake pointers; returns the status."""
    K, n = over.pop("K", 2), 2
    cfg = B.Config(K=K, inner=0, H=4, p=0.25, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01,
                   momentum=0.0, outer_lr=0.7, outer_momentum=0.9, outer_nesterov=1, precision=0, seed=1)
    ptr = over.pop("ptr", 0x10000)
    for k_, v_ in list(over.items()):
        if hasattr(cfg, k_):
            setattr(cfg, k_, over.pop(k_))
    kn = max(K, 1) * n
    mk = lambda base: C.cast((C.c_void_p * kn)(*[C.c_void_p(base + 0x1000 * i) for i in range(kn)]),
                             C.POINTER(C.c_void_p))
    bufs = B.Buffers(param=mk(ptr), grad=mk(ptr + 0x100000), master=None, m=mk(ptr + 0x200000),
                     v=mk(ptr + 0x300000), global_=mk(ptr + 0x400000), outer_mom=mk(ptr + 0x500000))
    for k_, v_ in over.items():
        setattr(bufs, k_, v_)
    ctx = C.c_void_p()
    numel = (C.c_uint64 * n)(8, 8)
    rc = P.lib().palsgd_init(C.byref(ctx), C.byref(cfg), n, numel, C.byref(bufs), None)
    assert not ctx.value or rc == 0
    return rc


@pytest.mark.parametrize("over", [
    dict(K=0), dict(K=65), dict(H=0), dict(p=-0.01), dict(p=1.01), dict(p=float("nan")),
    dict(inner=2), dict(precision=3), dict(outer_nesterov=2), dict(beta1=1.0), dict(eps=-1.0),
    dict(weight_decay=float("inf")), dict(v=None), dict(param=None), dict(outer_mom=None),
])
def test_init_rejects_bad_configuration_before_any_cuda_call(over):
    assert _fake_init(**over) == -1


def test_init_rejects_misaligned_pointer():
    assert _fake_init(ptr=0x10002) == -2


def test_null_context_and_null_outputs_are_rejected():
    L = P.lib()
    assert L.palsgd_init(None, None, 0, None, None, None) == -1
    assert L.palsgd_inner_step(None, 1e-3, 1.0, None) == -1
    assert L.palsgd_pseudo_sync(None, 1, 0.1, None) == -1
    assert L.palsgd_outer_sync(None, None) == -1
    assert L.palsgd_step(None, 1e-3, 1.0, None) == -1
    assert L.palsgd_get_counters(None, None, None, None, None, None) == -1
    assert L.palsgd_get_launch_count(None, None) == -1
    L.palsgd_destroy(None)      # accepted


def test_valid_arguments_without_a_gpu_fail_cleanly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    assert _fake_init() in (-3, -5)             # CUDA error, not a crash
    assert P.lib().palsgd_last_cuda_error(None) != b""


def test_missing_library_is_a_loud_error(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", tmp_path / "nope.so")
    with pytest.raises(ImportError):
        B.lib()


def test_later_entry_points_reject_a_null_context():
    L = P.lib()
    assert L.palsgd_ddp_step(None, 1e-3, None) == -1
    assert L.palsgd_set_grad_clip(None, 1.0) == -1
    assert L.palsgd_get_grad_norms(None, None, None, None) == -1
    assert L.palsgd_set_outer_lr(None, 0.5) == -1
    assert L.palsgd_cycle_capture(None, 1e-3, 1.0) == -1
    assert L.palsgd_cycle_launch(None, None) == -1
    assert L.palsgd_step_host(None, None, 1e-3, 1.0, None, None, None, None) == -1
    assert L.palsgd_set_tuning(None, 0, 0) == -1
    assert L.palsgd_get_layout(None, None, None, None) == -1
    assert L.palsgd_exchange_numel(None, None) == -1
    assert L.palsgd_set_worker_offset(None, 0) == -1
    assert L.palsgd_outer_partial(None, None, None) == -1
    assert L.palsgd_outer_finish(None, None, 1, None) == -1
    assert L.palsgd_global_from_exchange(None, None, 1, None) == -1
    assert L.palsgd_ddp_partial(None, None, None) == -1
    assert L.palsgd_ddp_finish(None, None, 1, 1e-3, None) == -1


@pytest.mark.parametrize("over", [dict(outer_opt=2), dict(outer_opt=1),                      # AdamW outer without outer_v
                                  dict(outer_opt=1, outer_beta1=1.0), dict(outer_opt=1, outer_eps=-1.0)])
def test_init_rejects_bad_outer_optimizer_settings(over):
    assert _fake_init(**over) == -1


def test_no_allocation_entry_point_validates_before_touching_the_gpu():
    L = P.lib()
    vp = C.c_void_p
    arr = lambda *a: C.cast((vp * len(a))(*[vp(x) for x in a]), C.POINTER(vp))
    numel = (C.c_uint64 * 1)(8)
    ok_ptrs = dict(param=arr(0x10000), master=None, global_=arr(0x20000), outer_mom=arr(0x30000))
    call = lambda K=1, prec=0, numel=numel, lr=0.7, mu=0.9, nest=1, **p: L.palsgd_outer_sync_noalloc(
        K, prec, 1, numel, p.get("param", ok_ptrs["param"]), p.get("master", None),
        p.get("global_", ok_ptrs["global_"]), p.get("outer_mom", ok_ptrs["outer_mom"]), lr, mu, nest, None)
    assert call(K=0) == -1 and call(K=65) == -1 and call(prec=2) == -1 and call(nest=2) == -1
    assert call(lr=float("nan")) == -1 and call(mu=-0.5) == -1
    assert call(prec=1) == -1                                            # mixed precision needs the masters
    assert call(param=arr(0)) == -1                                      # NULL slot pointer of a non-empty tensor
    assert call(param=arr(0x10002)) == -2                                # not aligned to the element size
    assert call(numel=(C.c_uint64 * 1)(8192 * 70000)) == -8              # tables beyond the fixed scratch
    assert call(numel=(C.c_uint64 * 1)(0)) == 0                          # nothing to do
