"""The N > 1 logic of bench.py on CPU: two gloo ranks reduce their timings with MAX and
form the whole-job value; the reference arm prints from rank 0 only."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r'''
import os, sys, json
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
ms = [10.0 + 5.0 * rank, 100.0 - 30.0 * rank]          # rank 1 is slower in the first, faster in the second
out = bench.max_over_ranks(ms, world)
val = bench.whole_job_value(world, 8, 1000, 4, out[0])
with open(os.path.join(sys.argv[2], f"rank{rank}.json"), "w") as f:      # one file per rank: stdout may interleave
    json.dump({"rank": rank, "max": out, "value": val}, f)
dist.barrier()
dist.destroy_process_group()
'''


def _torchrun(args, port=None):
    from conftest import free_port
    port = free_port()                  # whatever the caller asked for: a port that is free now
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port)] + args
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)


def test_timings_are_reduced_with_max_and_value_counts_every_rank(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    r = _torchrun([str(script), ROOT, str(tmp_path)], 29611)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.load(open(tmp_path / f"rank{k}.json")) for k in (0, 1)]
    assert sorted(l["rank"] for l in lines) == [0, 1]
    for l in lines:
        assert l["max"] == [15.0, 100.0]                               # slowest rank per entry
        assert l["value"] == pytest.approx(2 * 8 * 1000 * 4 / 15e-3)   # both ranks' work over the slowest time


SHARD_WORKER = r'''
import os, sys, json
sys.path.insert(0, sys.argv[1])
import numpy as np
import torch, torch.distributed as dist
import bench, workloads as W
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
cfg = W.get_config("c1_gptneo8m")
numel = [t.numel for t in cfg.tensors]
out = {}
for shard in (False, True):
    mine, lo, hi, seed_off, P_job = bench.rank_share(numel, rank, world, shard)
    x = W.init_params_host(cfg.tensors, cfg.param_seed + seed_off, cfg.init_std)[lo:hi]
    spans = [None] * world
    dist.all_gather_object(spans, (lo, hi, sum(mine), float(x[:3].sum()), seed_off, P_job))
    out["shard" if shard else "replica"] = spans
with open(os.path.join(sys.argv[2], f"share{rank}.json"), "w") as f:
    json.dump(out, f)
dist.barrier(); dist.destroy_process_group()
'''


def test_sharded_arm_gives_every_rank_its_slice_of_one_model(tmp_path):
    script = tmp_path / "share.py"
    script.write_text(SHARD_WORKER)
    r = _torchrun([str(script), ROOT, str(tmp_path)], 29613)
    assert r.returncode == 0, r.stderr[-2000:]
    sys.path.insert(0, ROOT)
    import workloads as W
    cfg = W.get_config("c1_gptneo8m")
    x = W.init_params_host(cfg.tensors, cfg.param_seed, cfg.init_std)
    for rank in (0, 1):
        d = json.load(open(tmp_path / f"share{rank}.json"))
        (lo0, hi0, n0, head0, so0, job0), (lo1, hi1, n1, head1, so1, job1) = d["shard"]
        assert lo0 == 0 and hi0 == lo1 and hi1 == cfg.P and n0 == hi0 - lo0 and n1 == hi1 - lo1   # a partition
        assert so0 == so1 == 0 and job0 == job1 == cfg.P                       # one model, strong scaling
        assert head0 == pytest.approx(float(x[:3].sum())) and head1 == pytest.approx(float(x[lo1:lo1 + 3].sum()))
        (a0, b0, m0, _, s0, j0), (a1, b1, m1, _, s1, j1) = d["replica"]
        assert (a0, b0, a1, b1) == (0, cfg.P, 0, cfg.P) and (s0, s1) == (0, 1) and j0 == j1 == 2 * cfg.P


def test_single_rank_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], 1) == [1.5, 2.5]
    assert bench.whole_job_value(1, 4, 10, 2, 1.0) == pytest.approx(80 / 1e-3)


def test_reference_arm_under_torchrun_prints_one_line_from_rank_zero():
    r = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "2", "--warmup", "0",
                   "--workload", "c0_flat_1m"], 29612)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = lines[0]
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0
