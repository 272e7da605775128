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
spec = bench.workload("cfg4", 3, rank)
print("RESULT", rank, ms, spec.seed, flush=True)
dist.destroy_process_group()
"""


def test_class_units_of_the_bench_workload():
    sys.path.insert(0, ROOT)
    import bench
    spec = bench.workload("cfg4", 100)
    u = bench.class_units(spec)
    assert u["small"] == [4096 * 800, 512 * 600 + 512 * 200] and u["warp"] == [4096 * 200, 64 * 200]
    assert u["mid"] == [0, 0] and u["large"] == [0, 0]
    assert sum(x[0] for x in u.values()) == 4_096_000
    assert bench.workload("cfg4", 3, 1).seed != bench.workload("cfg4", 3, 0).seed


def test_units_and_bytes_of_the_other_workloads():
    sys.path.insert(0, ROOT)
    import bench
    w = bench.workload("cfg4w")
    assert w.n_windows == 100 and bench.class_units(w)["large"] == [4_096_000, 1000]
    assert bench.kernel_units(w)["k_reduce_large"] == (4_096_000, 1000) and bench.kernel_units(w)["k_reduce_fused"] == (0, 0)
    s = bench.workload("cfg5")
    u = bench.class_units(s)
    assert s.n_windows == 50 and s.hang.window == 25
    assert u["small"] == [16_384 * 500, 2048 * 500] and u["warp"] == [16_384 * 250, 128 * 250]
    assert u["large"] == [16_384 * 250, 8 * 250] and u["mid"] == [1024 * 10, 10]
    # a reduce kernel's method bytes: values and flag per record, one row per group; the record index it also reads is overhead
    assert bench.algorithmic_bytes("k_reduce_fused", 1000, 10) == (34 * 1000 + 104 * 10, 4 * 1000)
    assert bench.algorithmic_bytes("k_seq_range", 1000, 10) == (8000, 0)
    assert bench.algorithmic_bytes("k_slot_scatter", 1000, 10) == (12000, 4000)


def test_ncu_traffic_goes_stale_with_the_kernel_source(monkeypatch):
    sys.path.insert(0, ROOT)
    import bench
    ent = bench.NCU_TRAFFIC["k_reduce_fused"]
    fresh = bench.sources_sha16(ent["files"]) == ent["sha16"]
    t = bench.ncu_traffic("k_reduce_fused", 1_000_000)
    assert (t is not None) == fresh
    if fresh:
        assert t == ent["bytes_per_record"] * 1_000_000
    monkeypatch.setitem(bench.NCU_TRAFFIC, "k_reduce_fused", dict(ent, sha16="0" * 16))
    assert bench.ncu_traffic("k_reduce_fused", 1_000_000) is None
    assert bench.ncu_traffic("k_plan", 5) is None


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
