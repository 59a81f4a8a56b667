"""The N > 1 plumbing of bench.py on CPU: two gloo ranks (replicas only, no data-path collective).

Checks the only cross-rank step the benchmark has -- the max-over-ranks of the timed region --
and that replicas get distinct seeded inputs while the reference arm stays on rank 0."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import numpy as np
import torch.distributed as dist
import bench
from paper_2607_27042_b200 import workloads as W
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist)          # rank 1 is the slow one
X, A, B = W.gaussian_like(16, 24, seed=0 + rank)             # replica inputs: seed + rank, as bench.py does
dist.barrier()
with open(os.path.join(%r, "rank%%d.json" %% rank), "w") as f:       # one file per rank: stdout lines can interleave
    json.dump({"rank": rank, "world": world, "ms": ms, "value": bench.job_value(16, 24, world, ms),
               "x00": float(X[0, 0])}, f)
dist.destroy_process_group()
"""


def test_two_gloo_ranks_agree_on_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % (ROOT, str(tmp_path)))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29571", OMP_NUM_THREADS="1")
    out = subprocess.run(
        [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
         "--master-addr", "127.0.0.1", "--master-port", "29571", str(script)],
        capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    rows = [json.load(open(tmp_path / ("rank%d.json" % r))) for r in range(2)]
    assert sorted(r["rank"] for r in rows) == [0, 1]
    assert all(r["ms"] == 15.0 for r in rows)                 # both report the max over ranks
    assert all(abs(r["value"] - 2 * 16 * 24 / 0.015) < 1e-6 for r in rows)
    assert rows[0]["x00"] != rows[1]["x00"]                   # distinct replicas


def test_reference_arm_runs_on_rank_zero_only(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")

    class A:
        config = 0; seed = 0; steps = 1; warmup = 0; ref_coords = 8
    bench.run_reference(A())
    assert capsys.readouterr().out == ""
