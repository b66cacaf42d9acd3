"""The measurement tools run end to end on a tiny case (they produce the published figures,
so they should not rot)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(args):
    r = subprocess.run([sys.executable] + args, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    return r.stdout


def test_sweep_prints_a_table_row_per_point():
    out = _run(["-m", "paper_2504_18454_b200.sweep", "--K", "4", "--logP", "20", "--p", "0,1", "--steps", "3"])
    rows = [l for l in out.splitlines() if l.startswith("| 4 | 2^20")]
    assert len(rows) == 2 and "inner GB/s" in out


def test_bench_line_has_the_contract_keys():
    out = _run(["bench.py", "--workload", "c0_flat_1m", "--steps", "16", "--warmup", "3"])
    d = json.loads([l for l in out.splitlines() if l.startswith("{")][-1])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks"):
        assert key in d, key
    assert d["roofline"]["bound"] == "hbm" and d["roofline"]["achieved"] > 0 and d["gpu_launches"] == 16 + 2
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] > 0
    assert d["config"]["workload"] == "c0_flat_1m" and d["value"] > 0
    for part in ("partial", "finish", "ddp_partial", "ddp_finish"):
        assert d["outer_split"][part]["achieved"] > 0


def test_outer_sync_is_timed_even_when_no_sync_falls_inside_the_step_loop():
    # 4 timed steps with H = 8: the step loop contains no outer sync, yet the metric's
    # "per outer_sync" half must be measured
    out = _run(["bench.py", "--workload", "c0_flat_1m", "--steps", "4", "--warmup", "3", "--no-e2e",
                "--no-cpu-baseline", "--no-graph", "--no-ddp"])
    d = json.loads([l for l in out.splitlines() if l.startswith("{")][-1])
    ro = d["roofline_outer"]
    assert ro["launches_inside_step_loop"] == 0 and ro["launches_timed_alone"] == 8 and ro["launches"] == 8
    for key in ("achieved", "frac", "frac_of_nominal_peak", "avg_ms", "alg_bytes_per_launch", "params_per_s"):
        assert ro[key] is not None and ro[key] > 0, key
    assert ro["alg_bytes_per_launch"] == (8 * 4 + 16) * (1 << 20)
    assert d["cycle"]["H"] == 8 and d["cycle"]["ms_per_step"] > d["roofline"]["avg_ms"]
    assert d["gpu_launches"] == 4


@pytest.mark.parametrize("layout", ["separate", "misaligned"])
def test_bench_runs_on_the_ragged_layouts(layout):
    out = _run(["bench.py", "--workload", "c1_gptneo8m", "--steps", "4", "--warmup", "3", "--layout", layout,
                "--no-cpu-baseline", "--no-graph", "--e2e-steps", "2"])
    d = json.loads([l for l in out.splitlines() if l.startswith("{")][-1])
    assert d["config"]["layout"] == layout
    assert d["config"]["n_segments"] == (99 if layout == "separate" else 1)
    assert d["roofline"]["achieved"] > 0 and d["roofline_outer"]["achieved"] > 0 and d["e2e"]["value"] > 0


def test_default_layout_run_also_times_the_ragged_layout():
    out = _run(["bench.py", "--workload", "c1_gptneo8m", "--steps", "4", "--warmup", "3", "--no-e2e",
                "--no-cpu-baseline", "--no-graph", "--no-ddp"])
    d = json.loads([l for l in out.splitlines() if l.startswith("{")][-1])
    rg = d["ragged_layout"]
    assert d["config"]["layout"] == "arena" and d["config"]["n_segments"] == 1
    assert rg["layout"] == "separate" and rg["n_segments"] == 99
    assert rg["roofline"]["launches"] == 16 and rg["roofline"]["achieved"] > 0 and rg["roofline"]["traffic"] is None
    assert rg["roofline_outer"]["launches"] == 4 and rg["roofline_outer"]["achieved"] > 0
    assert d["gpu_launches"] == 4                      # the extra region is not part of the timed step loop


@pytest.mark.parametrize("launcher", ["plain", "torchrun"])
def test_bench_workers_mode_runs_with_one_rank(launcher):
    from conftest import free_port
    # the paper's deployment (workers spread over the ranks, outer sync around an all-reduce) with the one rank a
    # single GPU allows: plain (no process group) and under torchrun (NCCL process group of one rank)
    tail = ["bench.py", "--gpus", "1", "--workers", "--workload", "c0_flat_1m", "--steps", "16", "--warmup", "3"]
    head = [] if launcher == "plain" else ["-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "1",
                                           "--master-addr", "127.0.0.1", "--master-port", str(free_port())]
    out = _run(head + tail)
    d = json.loads([l for l in out.splitlines() if l.startswith("{")][-1])
    assert d["scaling"] == "strong" and d["n_gpus"] == 1 and d["value"] > 0
    ex = d["outer_exchange"]
    assert ex["syncs"] == 2 and ex["partial"]["achieved"] > 0 and ex["finish"]["achieved"] > 0     # H = 8
    assert ex["all_reduce"]["bytes"] == 4 * (1 << 20)
    assert ex["all_reduce"]["backend"] == ("nccl" if launcher == "torchrun" else "none (one rank)")
    assert d["roofline"]["achieved"] > 0 and d["gpu_launches"] == 16 + 2 * 2
