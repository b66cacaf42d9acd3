"""The measurement tools run end to end on a tiny case (they are how the figures in the
design notes were produced, so they should not rot)."""
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


def test_tune_times_every_kernel():
    out = _run(["-m", "paper_2504_18454_b200.tune", "c0_flat_1m", "--variants", "0,18", "--steps", "4",
                "--outer-dynamic", "0,2"])
    for needle in ("inner variant=0", "inner variant=18", "grad-norm pass (per worker)", "grad-norm pass (ddp)",
                   "outer slice=1024 variant=2", "ddp slice=1024 variant=1"):
        assert needle in out, needle


def test_bench_line_has_the_contract_keys():
    out = _run(["bench.py", "--workload", "c0_flat_1m", "--steps", "16", "--warmup", "3"])
    d = json.loads([l for l in out.splitlines() if l.startswith("{")][-1])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks"):
        assert key in d, key
    assert d["roofline"]["bound"] == "hbm" and d["roofline"]["achieved"] > 0 and d["gpu_launches"] == 16 + 2
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] > 0
    assert d["config"]["workload"] == "c0_flat_1m" and d["value"] > 0
