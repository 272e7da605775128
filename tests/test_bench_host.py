"""Host-side logic of bench.py on CPU: per-rank workloads, unit accounting, and the max-over-ranks
timing reduction over a world_size-2 gloo group."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
import torch, torch.distributed as dist
import bench
rank = int(os.environ["RANK"])
dist.init_process_group("gloo")
ms = bench.max_over_ranks(10.0 + 5.0 * rank, torch.device("cpu"))
spec = bench.workload(3, rank)
print("RESULT", rank, ms, spec.seed, flush=True)
dist.destroy_process_group()
"""


def test_class_units_of_the_bench_workload():
    sys.path.insert(0, ROOT)
    import bench
    spec = bench.workload(100)
    u = bench.class_units(spec)
    assert u["small"] == [4096 * 800, 512 * 600 + 512 * 200] and u["warp"] == [4096 * 200, 64 * 200]
    assert u["mid"] == [0, 0] and u["large"] == [0, 0]
    assert sum(x[0] for x in u.values()) == 4_096_000
    assert bench.workload(3, 1).seed != bench.workload(3, 0).seed


def test_max_over_ranks_with_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", LOCAL_RANK=str(r), MASTER_ADDR="127.0.0.1", MASTER_PORT="29613")
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    res = sorted(line.split() for o in outs for line in o.splitlines() if line.startswith("RESULT"))
    assert len(res) == 2
    assert float(res[0][2]) == 15.0 and float(res[1][2]) == 15.0          # both ranks see the slower rank's time
    assert res[0][3] != res[1][3]                                         # every rank analyses its own trace
