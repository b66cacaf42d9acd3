"""GPU parity, small cases: the CUDA library against the CPU oracle, element by
element, over shapes that span several chunks and ragged tails, both optimizers,
both precisions, all three buffer layouts, and the degenerate settings."""
import numpy as np
import pytest
import torch

import paper_2504_18454_b200 as pkg
import workloads as W
from workloads.configs import WorkloadConfig
from _harness import GpuRun, compare_state, make_oracle

pytestmark = pytest.mark.gpu

RAGGED = [1, 3, 7, 1001, 4095, 4096, 4097, 0, 5, 12289, 8]     # > 6 chunks, odd tails, an empty tensor


def _cfg(numel, **kw):
    base = dict(name="t", shape=lambda: [], K=4, H=4, p=0.25, eta=16.0, lr=1e-3, T=10)
    base.update(kw)
    return WorkloadConfig(**base)


def _x0(K, P, seed=1, same=False):
    rng = np.random.default_rng(seed)
    if same:
        return np.tile((rng.standard_normal(P) * 0.02).astype(np.float32), (K, 1))
    return (rng.standard_normal((K, P)) * 0.02).astype(np.float32)


def _grads(cfg, P, t):
    g = np.stack([W.grads_host(P, cfg.grad_seed, t, k, cfg.grad_std) for k in range(cfg.K)])
    return W.bf16_bits_from_f32_host(g) if cfg.precision == 1 else g


def _run_both(cfg, numel, layout, T=None, x0=None, check_every_step=True):
    P = int(sum(numel))
    x0 = _x0(cfg.K, P) if x0 is None else x0
    gpu = GpuRun(cfg, x0, numel=numel, layout=layout)
    orc = make_oracle(cfg, x0)
    compare_state(gpu.state(), orc, exact=True)                   # init: mean, zeros, bf16 copy
    for t in range(T if T is not None else cfg.T):
        g = _grads(cfg, P, t)
        gpu.set_grads(g)
        gpu.step(cfg.lr, cfg.eta)
        orc.step(g, cfg.lr, cfg.eta)
        if check_every_step:
            c = gpu.counters()
            assert c["t"] == orc.t and c["n_outer"] == orc.n_outer
            assert c["s"] == [int(v) for v in orc.s]              # bit-exact integer state
            assert c["last_b"] == [int(v) for v in orc.last_b]
    rep = compare_state(gpu.state(), orc, exact=True)
    assert gpu.guards_intact()
    return gpu, orc, rep


@pytest.mark.parametrize("layout", ["arena", "separate", "misaligned"])
@pytest.mark.parametrize("inner,precision", [(0, 0), (1, 0), (0, 1), (1, 1)])
def test_ragged_tensor_list_matches_oracle(layout, inner, precision):
    cfg = _cfg(RAGGED, inner=inner, precision=precision, momentum=0.9 if inner else 0.0,
               weight_decay=1e-4 if inner else 0.01)
    _run_both(cfg, RAGGED, layout)


@pytest.mark.parametrize("precision", [0, 1])
@pytest.mark.parametrize("numel", [[50], [64, 3], [191], [190, 9], [8192 + 70, 5, 200]])
def test_long_scalar_head_in_front_of_a_list_one_element_off_a_256_element_grid(numel, precision):
    # rows a multiple of 256 elements apart: every buffer starts 64 + 1 elements behind a multiple of 256 elements, and
    # the library peels the 191 elements that put all of them back on one (more than some of these lists hold) instead
    # of the 3 or 7 that 16 bytes would need
    cfg = _cfg(numel, K=3, H=3, T=7, precision=precision)
    P = int(sum(numel))
    x0 = _x0(cfg.K, P)
    gpu, orc = GpuRun(cfg, x0, numel=numel, layout="misaligned", row_align=256), make_oracle(cfg, x0)
    lay, head = gpu.lib.get_layout(), 191
    assert lay["n_segments"] == 1 and lay["n_chunks"] == 1 + (0 if P <= head else -(-(P - head) // lay["chunk_elems"]))
    gpu.set_grad_clip(0.05); orc.set_grad_clip(0.05)
    for t in range(2):                                            # the DDP kernel and the norm pass over the same pieces
        g = _grads(cfg, P, t)
        gpu.set_grads(g); gpu.ddp_step(cfg.lr); orc.ddp_step(g, cfg.lr)
    for t in range(2, 2 + cfg.T):
        g = _grads(cfg, P, t)
        gpu.set_grads(g); gpu.step(cfg.lr, cfg.eta); orc.step(g, cfg.lr, cfg.eta)
        assert gpu.counters()["last_b"] == [int(v) for v in orc.last_b]
    compare_state(gpu.state(), orc, exact=True)
    assert gpu.counters()["n_outer"] == orc.n_outer >= 2 and gpu.guards_intact()


@pytest.mark.parametrize("layout,precision", [("separate", 0), ("separate", 1), ("arena", 1)])
def test_thousands_of_small_tensors(layout, precision):
    # one segment per tensor when every tensor is its own allocation: 3000 segments, most of them far smaller than
    # a work item, some empty, a few spanning several chunks
    rng = np.random.default_rng(17)
    numel = [int(n) for n in rng.integers(0, 300, size=3000)]
    for j in (5, 1500, 2999):
        numel[j] = 8192 * 2 + 77
    cfg = _cfg(numel, K=2, H=2, T=4, precision=precision)
    gpu, orc, _ = _run_both(cfg, numel, layout, check_every_step=False)
    lay = gpu.lib.get_layout()
    nonempty = [n > 0 for n in numel]
    runs = sum(1 for j, ne in enumerate(nonempty) if ne and (j == 0 or not nonempty[j - 1]))
    # (packed: an empty tensor reports a NULL pointer, which ends a run of adjacent tensors)
    if layout == "separate":     # (two allocations that happen to sit back to back in every buffer are fused: rare)
        assert 0.98 * sum(nonempty) <= lay["n_segments"] <= sum(nonempty)
    else:
        assert lay["n_segments"] == runs
    gpu.set_grad_clip(0.01); orc.set_grad_clip(0.01)
    P_ = int(sum(numel))
    for t in range(4, 6):
        g = _grads(cfg, P_, t)
        gpu.set_grads(g); gpu.step(cfg.lr, cfg.eta); orc.step(g, cfg.lr, cfg.eta)
    compare_state(gpu.state(), orc, exact=True)
    assert gpu.guards_intact()


@pytest.mark.parametrize("K", [1, 2, 3, 8, 32, 64])
def test_worker_counts(K):
    numel = [4096 * 2 + 13]
    cfg = _cfg(numel, K=K, H=3, T=7)
    _run_both(cfg, numel, "arena")


@pytest.mark.parametrize("numel", [[1], [3], [7], [4095], [4097], [0, 0, 2]])
def test_tiny_and_edge_sizes(numel):
    _run_both(_cfg(numel, K=3, H=2, T=5), numel, "separate")
    _run_both(_cfg(numel, K=3, H=2, T=5, precision=1), numel, "arena")


@pytest.mark.parametrize("p", [0.0, 1.0, 0.5])
def test_extreme_probabilities(p):
    numel = [5000]
    gpu, orc, _ = _run_both(_cfg(numel, p=p, H=4, T=8), numel, "arena")
    c = gpu.counters()
    if p == 0.0:
        assert c["s"] == [8] * 4             # never pulls: DiLoCo
    if p == 1.0:
        assert c["s"] == [0] * 4             # always pulls


@pytest.mark.parametrize("precision", [0, 1])
def test_zero_step_size_and_zero_mixing_rate(precision):
    numel = [5000]
    # eta = 0: the pull coefficient is 0, a pulling worker keeps its model (and takes no gradient step)
    gpu, orc, _ = _run_both(_cfg(numel, eta=0.0, p=0.5, H=4, T=8, precision=precision), numel, "arena")
    # alpha = 0: the gradient branch moves the moments only
    x0 = _x0(4, 5000, same=True)
    gpu, orc, _ = _run_both(_cfg(numel, lr=0.0, p=0.5, H=4, T=3, precision=precision), numel, "arena", x0=x0)
    st = gpu.state()
    assert np.array_equal(st["x"], x0) and np.any(st["m"] != 0)


def test_plain_averaging_outer_and_momentum_without_nesterov():
    numel = [9000]
    _run_both(_cfg(numel, outer_lr=1.0, outer_momentum=0.0, outer_nesterov=False, H=3, T=6), numel, "arena")
    _run_both(_cfg(numel, outer_lr=0.5, outer_momentum=0.8, outer_nesterov=False, H=3, T=6), numel, "arena")


def test_h_equal_one_and_t_not_multiple_of_h():
    numel = [4099]
    _run_both(_cfg(numel, H=1, T=4), numel, "arena")
    _run_both(_cfg(numel, H=5, T=7), numel, "arena")


def test_slots_that_differ_at_start_get_the_fixed_order_mean():
    numel = [6000]
    cfg = _cfg(numel, K=5)
    _run_both(cfg, numel, "arena", x0=_x0(5, 6000, seed=3, same=False), T=5)


def test_large_pull_coefficient_is_not_clamped():
    numel = [3000]
    _run_both(_cfg(numel, eta=400.0, p=0.25, T=6), numel, "arena")      # beta = 1.6


def test_separate_entry_points_inner_pull_outer():
    numel = RAGGED
    P = sum(numel)
    for precision in (0, 1):
        cfg = _cfg(numel, precision=precision, H=10**6)
        x0 = _x0(cfg.K, P, seed=9)
        gpu, orc = GpuRun(cfg, x0, numel=numel), make_oracle(cfg, x0)
        for t in range(3):
            g = _grads(cfg, P, t)
            gpu.set_grads(g); gpu.inner_step(cfg.lr, cfg.eta); orc.inner_step(g, cfg.lr, cfg.eta)
        gpu.pseudo_sync(0b0101, 0.3); orc.pseudo_sync(0b0101, 0.3)
        compare_state(gpu.state(), orc, exact=True)
        c = gpu.counters()
        assert c["t"] == 3 and c["n_outer"] == 0 and c["s"] == [int(v) for v in orc.s]
        gpu.outer_sync(); orc.outer_sync()
        st = gpu.state()
        compare_state(st, orc, exact=True)
        for k in range(cfg.K):                                    # consensus, bitwise
            assert np.array_equal(st["x"][k], st["xg"])
        assert gpu.counters()["n_outer"] == 1
        gpu.pseudo_sync(0, 0.3)                                   # empty mask: no-op
        with pytest.raises(Exception):
            gpu.pseudo_sync(1 << cfg.K, 0.3)                      # bit beyond K


def test_checkpoint_resume_is_bit_exact():
    numel = [10000]
    cfg = _cfg(numel, H=4)
    P = 10000
    x0 = _x0(cfg.K, P, same=True)
    a = GpuRun(cfg, x0, numel=numel)
    for t in range(8):
        a.set_grads(_grads(cfg, P, t)); a.step(cfg.lr, cfg.eta)
    want = a.state()
    b = GpuRun(cfg, x0, numel=numel)
    for t in range(4):
        b.set_grads(_grads(cfg, P, t)); b.step(cfg.lr, cfg.eta)
    saved, cnt = b.state(), b.counters()
    c = GpuRun(cfg, x0, numel=numel)                              # fresh context, restore, continue
    for name, key in (("param", "x"), ("m", "m"), ("v", "v")):
        c._write(name, saved[key])
    c._write("global_", saved["xg"][None]); c._write("outer_mom", saved["u"][None])
    c.lib.set_counters(cnt["t"], cnt["s"], cnt["n_outer"], c.stream)
    for t in range(4, 8):
        c.set_grads(_grads(cfg, P, t)); c.step(cfg.lr, cfg.eta)
    got = c.state()
    for k in want:
        assert np.array_equal(want[k], got[k]), k
    assert c.counters() == a.counters()


def test_run_to_run_determinism_and_launch_shape_independence():
    numel = RAGGED
    P = sum(numel)
    cfg = _cfg(numel, K=8, H=3, T=6)
    x0 = _x0(cfg.K, P, same=True)
    outs = []
    for caps in (None, None, (7, 3), (148 * 4, 148)):
        r = GpuRun(cfg, x0, numel=numel)
        if caps:
            r.lib.set_tuning(0, caps[0]); r.lib.set_tuning(1, caps[1])
        for t in range(cfg.T):
            r.set_grads(_grads(cfg, P, t)); r.step(cfg.lr, cfg.eta)
        outs.append(r.state())
        assert r.lib.get_launch_count() == 1 + cfg.T + cfg.T // cfg.H   # init + inner + outer
    for o in outs[1:]:
        for k in outs[0]:
            assert np.array_equal(outs[0][k], o[k]), k


@pytest.mark.parametrize("variant,cap", [(0, 0), (0, 5), (18, 0), (18, 7)])
@pytest.mark.parametrize("inner,precision", [(0, 0), (1, 0), (0, 1), (1, 1)])
def test_every_launch_form_of_the_inner_kernel_matches_oracle(variant, cap, inner, precision):
    # 0: persistent grid that draws its work items from a queue; 18: one CTA per item; a capped grid
    # strides over the items.  "misaligned": every buffer one element off 16-byte alignment, so each
    # segment starts with a few elements on the scalar path and continues on the vector path
    numel = [4096 * 37 + 11, 5, 4096 * 2, 1001]
    P = sum(numel)
    cfg = _cfg(numel, K=5, H=3, T=7, p=0.3, inner=inner, precision=precision,
               momentum=0.9 if inner else 0.0)
    x0 = _x0(cfg.K, P, seed=5)
    for layout in ("arena", "separate", "misaligned"):
        gpu, orc = GpuRun(cfg, x0, numel=numel, layout=layout), make_oracle(cfg, x0)
        gpu.lib.set_tuning(2, variant); gpu.lib.set_tuning(0, cap)
        for t in range(cfg.T):
            g = _grads(cfg, P, t)
            gpu.set_grads(g); gpu.step(cfg.lr, cfg.eta); orc.step(g, cfg.lr, cfg.eta)
        compare_state(gpu.state(), orc, exact=True)
        c = gpu.counters()
        assert c["s"] == [int(v) for v in orc.s] and c["t"] == cfg.T
        assert gpu.guards_intact()


def test_step_host_moves_gradients_and_results_through_host_buffers():
    numel = [5000, 37, 4096]
    P = sum(numel)
    for precision in (0, 1):
        cfg = _cfg(numel, precision=precision, H=2)
        x0 = _x0(cfg.K, P, same=True)
        gpu, orc = GpuRun(cfg, x0, numel=numel, layout="separate"), make_oracle(cfg, x0)
        gdt = torch.int16 if precision else torch.float32
        hg = torch.empty((cfg.K, P), dtype=gdt).pin_memory()
        hx = torch.empty(P, dtype=torch.float32).pin_memory()
        hb = torch.zeros(cfg.K, dtype=torch.uint8).pin_memory()
        starts = np.concatenate([[0], np.cumsum(numel)])
        es = hg.element_size()
        gp = gpu.lib.make_ptr_array([hg.data_ptr() + (k * P + int(starts[j])) * es
                                     for k in range(cfg.K) for j in range(len(numel))])
        xp = gpu.lib.make_ptr_array([hx.data_ptr() + int(starts[j]) * 4 for j in range(len(numel))])
        for t in range(4):
            g = _grads(cfg, P, t)
            hg.copy_(torch.from_numpy(g.view(np.int16) if precision else g))
            synced = gpu.lib.step_host(gp, cfg.lr, cfg.eta, xp, hb.data_ptr(), gpu.stream)
            orc.step(g, cfg.lr, cfg.eta)
            assert synced == ((t + 1) % 2 == 0)
            assert hb.tolist() == [int(v) for v in orc.last_b]
            if synced:
                assert np.array_equal(hx.numpy(), orc.xg)
        compare_state(gpu.state(), orc, exact=True)


def test_step_host_transfers_no_gradient_for_workers_that_pull_and_splits_the_step_per_worker():
    numel = [6000, 9]
    P = sum(numel)
    cfg = _cfg(numel, K=6, p=0.5, H=100)
    x0 = _x0(cfg.K, P, same=True)
    gpu, orc = GpuRun(cfg, x0, numel=numel, layout="arena"), make_oracle(cfg, x0)
    hg = torch.empty((cfg.K, P), dtype=torch.float32).pin_memory()
    starts = np.concatenate([[0], np.cumsum(numel)])
    gp = gpu.lib.make_ptr_array([hg.data_ptr() + (k * P + int(starts[j])) * 4
                                 for k in range(cfg.K) for j in range(len(numel))])
    launches = gpu.lib.get_launch_count()
    for t in range(6):
        marker = np.full((cfg.K, P), 1000.0 + t, dtype=np.float32)
        gpu.set_grads(marker)                                     # what the device buffers held before the call
        g = _grads(cfg, P, t)
        hg.copy_(torch.from_numpy(g))
        # pulling workers need no gradient at all: their host pointers may be NULL
        import paper_2504_18454_b200 as PL
        pulls = [PL.decision(cfg.decision_seed, t, k, cfg.p) for k in range(cfg.K)]
        gp_t = gpu.lib.make_ptr_array([0 if pulls[k] else hg.data_ptr() + (k * P + int(starts[j])) * 4
                                       for k in range(cfg.K) for j in range(len(numel))])
        gpu.lib.step_host(gp_t if t % 2 else gp, cfg.lr, cfg.eta, None, 0, gpu.stream)
        orc.step(g, cfg.lr, cfg.eta)
        assert pulls == [int(v) for v in orc.last_b]
        on_device = gpu._read("grad")
        for k in range(cfg.K):
            want = marker[k] if orc.last_b[k] else g[k]           # pulled: untouched; gradient step: copied
            assert np.array_equal(on_device[k], want), (t, k)
    compare_state(gpu.state(), orc, exact=True)
    assert gpu.lib.get_launch_count() - launches == 6 * cfg.K     # one launch per worker and step
    assert gpu.counters()["s"] == [int(v) for v in orc.s]


@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("precision", [0, 1])
def test_step_host_with_many_small_tensors_gathers_them_in_one_launch_per_worker(pinned, precision):
    # one allocation per tensor on the device, 60 small tensors: from pinned memory a worker's small copies are
    # performed by one launch of the gather kernel (plus the copy engine for the large tensor and for sources off
    # 16-byte alignment); from pageable memory everything goes through the copy engine.  Same results either way.
    rng = np.random.default_rng(3)
    numel = [int(n) for n in rng.choice([8, 64, 256, 768, 1000, 3072], size=60)] + [7, 300000, 0, 5, 128]
    P = sum(numel)
    cfg = _cfg(numel, K=3, p=0.3, H=2, precision=precision)
    x0 = _x0(cfg.K, P, same=True)
    gpu, orc = GpuRun(cfg, x0, numel=numel, layout="separate"), make_oracle(cfg, x0)
    gdt = torch.bfloat16 if precision else torch.float32
    hg = torch.empty((cfg.K, P), dtype=gdt)
    hg = hg.pin_memory() if pinned else hg
    es = hg.element_size()
    starts = np.concatenate([[0], np.cumsum(numel)])
    gp = gpu.lib.make_ptr_array([hg.data_ptr() + (k * P + int(starts[j])) * es
                                 for k in range(cfg.K) for j in range(len(numel))])
    import paper_2504_18454_b200 as PL
    launches, expected = gpu.lib.get_launch_count(), 0
    for t in range(4):
        g = _grads(cfg, P, t)
        src = torch.from_numpy(g.view(np.int16)).view(torch.bfloat16) if precision else torch.from_numpy(g)
        hg.copy_(src)
        gpu.lib.step_host(gp, cfg.lr, cfg.eta, None, 0, gpu.stream)
        orc.step(g, cfg.lr, cfg.eta)
        takes_gradient = [1 - PL.decision(cfg.decision_seed, t, k, cfg.p) for k in range(cfg.K)]
        expected += cfg.K + (sum(takes_gradient) if pinned else 0) + (1 if (t + 1) % cfg.H == 0 else 0)
        on_device = gpu._read("grad")
        for k in range(cfg.K):
            if takes_gradient[k]:
                assert np.array_equal(on_device[k], g[k]), (t, k)
    compare_state(gpu.state(), orc, exact=True)
    # (a worker whose small copies are mostly off 16-byte alignment on the host keeps to the copy engine)
    got, plain = gpu.lib.get_launch_count() - launches, 4 * cfg.K + 2
    assert plain < got <= expected if pinned else got == expected == plain
    assert gpu.guards_intact()


def test_step_host_gather_table_grows_inside_one_call():
    # worker 0's host row has 10 small tensors on 16-byte boundaries and 300 off them, worker 1's row the other way
    # round, so the pinned table sized after worker 0 is too small for worker 1 and has to grow in mid-call
    numel = [16] * 10 + [1] + [16] * 300
    P = sum(numel)
    cfg = _cfg(numel, K=3, p=0.0, H=2, inner=1, momentum=0.9)
    x0 = _x0(cfg.K, P, same=True)
    gpu, orc = GpuRun(cfg, x0, numel=numel, layout="separate"), make_oracle(cfg, x0)
    pitch, shift = (P + 8 + 3) // 4 * 4, [0, 3, 0]                              # elements; worker 1's row starts 12 bytes late
    hg = torch.empty(cfg.K * pitch, dtype=torch.float32).pin_memory()
    assert hg.data_ptr() % 16 == 0 and pitch % 4 == 0
    rows = [hg[k * pitch + shift[k]: k * pitch + shift[k] + P] for k in range(cfg.K)]
    starts = np.concatenate([[0], np.cumsum(numel)])
    gp = gpu.lib.make_ptr_array([rows[k].data_ptr() + int(starts[j]) * 4 for k in range(cfg.K) for j in range(len(numel))])
    launches = gpu.lib.get_launch_count()
    for t in range(3):
        g = _grads(cfg, P, t)
        for k in range(cfg.K):
            rows[k].copy_(torch.from_numpy(g[k]))
        gpu.lib.step_host(gp, cfg.lr, cfg.eta, None, 0, gpu.stream)
        orc.step(g, cfg.lr, cfg.eta)
        assert np.array_equal(gpu._read("grad"), g)
    compare_state(gpu.state(), orc, exact=True)
    assert gpu.lib.get_launch_count() - launches == 3 * (cfg.K + cfg.K) + 1      # inner + gather per worker; one sync
    assert gpu.guards_intact()


def test_step_host_validates_the_result_pointers_before_anything_is_enqueued():
    # a NULL entry in h_global on a step that ends with an outer sync: EINVAL, and nothing has moved
    numel = [3000, 40]
    P = sum(numel)
    cfg = _cfg(numel, H=2)
    x0 = _x0(cfg.K, P, same=True)
    gpu = GpuRun(cfg, x0, numel=numel, layout="separate")
    hg = torch.zeros((cfg.K, P), dtype=torch.float32).pin_memory()
    hx = torch.empty(P, dtype=torch.float32).pin_memory()
    starts = np.concatenate([[0], np.cumsum(numel)])
    gp = gpu.lib.make_ptr_array([hg.data_ptr() + (k * P + int(starts[j])) * 4
                                 for k in range(cfg.K) for j in range(len(numel))])
    good = gpu.lib.make_ptr_array([hx.data_ptr() + int(starts[j]) * 4 for j in range(len(numel))])
    bad = gpu.lib.make_ptr_array([hx.data_ptr(), 0])
    assert gpu.lib.step_host(gp, cfg.lr, cfg.eta, bad, 0, gpu.stream) is False     # t = 1: no sync, pointers unused
    before, launches = gpu.state(), gpu.lib.get_launch_count()
    with pytest.raises(Exception) as e:
        gpu.lib.step_host(gp, cfg.lr, cfg.eta, bad, 0, gpu.stream)                 # t = 2 would sync
    assert getattr(e.value, "status", None) == -1
    c = gpu.counters()                                                             # host and device agree: OK
    assert c["t"] == 1 and c["n_outer"] == 0 and gpu.lib.get_launch_count() == launches
    after = gpu.state()
    for key in before:
        assert np.array_equal(before[key], after[key]), key
    assert gpu.lib.step_host(gp, cfg.lr, cfg.eta, good, 0, gpu.stream) is True     # the context is still usable
    assert gpu.counters()["n_outer"] == 1


@pytest.mark.parametrize("layout", ["arena", "separate", "misaligned"])
@pytest.mark.parametrize("precision", [0, 1])
def test_the_host_only_plan_agrees_with_what_init_built(layout, precision):
    numel = [8192 * 2 + 5, 7, 0, 100, 300]
    cfg = _cfg(numel, precision=precision)
    gpu = GpuRun(cfg, _x0(cfg.K, sum(numel)), numel=numel, layout=layout, row_align=256)
    addr = lambda name: [[int(t.data_ptr()) for t in row] for row in gpu.views[name]]
    plan = pkg.plan_layout(K=cfg.K, numel=numel, precision=precision, inner=cfg.inner, param=addr("param"),
                         grad=addr("grad"), m=addr("m"), v=addr("v"), master=addr("master") if precision else None,
                         global_=addr("global_")[0], outer_mom=addr("outer_mom")[0])
    built = gpu.lib.get_layout()
    assert {k: plan[k] for k in built} == built
    assert sum(n for _, n, _ in plan["segments"]) <= len(numel) and all(-1 <= h < 256 for _, _, h in plan["segments"])


def test_layout_report_counts_segments_and_chunks():
    numel = [8192 * 2 + 5, 7, 0, 100]
    cfg = _cfg(numel, inner=1, momentum=0.9)                     # 8192-element chunks
    x0 = _x0(cfg.K, sum(numel))
    # packed: the empty tensor (a NULL pointer) ends the first run of adjacent tensors
    packed = GpuRun(cfg, x0, numel=numel, layout="arena").lib.get_layout()
    assert packed == {"n_segments": 2, "n_chunks": 4, "chunk_elems": 8192}
    # one element off, rows a multiple of 256 elements apart: per segment a scalar head up to the next multiple of 256
    # elements (191 and 179 of them), then aligned chunks: 1 + 2 and 1 + 0
    shifted = GpuRun(cfg, x0, numel=numel, layout="misaligned", row_align=256).lib.get_layout()
    assert shifted["n_segments"] == 2 and shifted["n_chunks"] == 4
    # rows 8 elements (mod 128) apart: no common boundary beyond 16 bytes, heads of 3 elements: 1 + 3 and 1 + 1
    shifted = GpuRun(cfg, _x0(cfg.K, sum(numel) + 8), numel=numel + [8], layout="misaligned").lib.get_layout()
    assert shifted["n_segments"] == 2 and shifted["n_chunks"] == 6
    apart = GpuRun(cfg, x0, numel=numel, layout="separate").lib.get_layout()
    assert apart["n_segments"] == 3 and apart["n_chunks"] == 5
