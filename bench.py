"""Benchmark of the CCL-D analyzer hot path: trace records analysed per second at 4,096 ranks.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--windows NW]

A step is one pass of the whole hot path (group-by, per-op reductions, median/MAD flags, votes,
window decision) over the streaming slow-mix workload: 4,096 ranks (TP8 x PP8 x DP64), NW windows
of 1,000 ops per rank (NW = 100: 409.6 M records, 18.4 GB of SoA columns resident in HBM).
For N > 1 (under torch.distributed.run) every rank analyses its own trace on its own GPU: the path
has no exchange step, so the ranks only meet at the timing barrier.

--impl reference times the CPU oracle (one host core) on a bounded sample of the same workload.
Rank 0 prints one JSON line.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "trace records analyzed/sec at 4,096 ranks"
UNIT = "records/s"
REC_BYTES = 45            # 3 x u32 keys, u8 op, u64 bytes, 2 x i64 times, 2 x u32 rate columns
ROW_BYTES = 104           # one per-op row
HBM_FALLBACK_GBS = 6650.0
# DRAM traffic per record (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture divided by the records of the
# captured launch; 5-window case, 20.48 M records, see profiles/). Traffic grows in proportion to the records, so a
# launch's traffic is this figure times its records. Set an entry to None whenever its kernel changes.
NCU_TRAFFIC_PER_RECORD = {"k_reduce_fused": (784.674560e6 + 243.086848e6) / 20.48e6}


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--windows", type=int, default=100, help="windows of 1,000 ops per rank resident on the GPU")
    ap.add_argument("--e2e-windows", type=int, default=10, help="windows per end-to-end step (host buffers)")
    ap.add_argument("--cpu-windows", type=int, default=10, help="windows the CPU oracle is timed on")
    ap.add_argument("--mix", default="all", choices=sorted(MIXES), help="all: the cfg4 workload; tp_pp / dp: only its 8-rank or only its 64-rank "
                    "communicators (timing one path of the fused kernel; the headline number is --mix all)")
    ap.add_argument("--rate-windows", type=int, default=2, help="windows whose raw probe samples are turned into rate columns (0 = skip)")
    return ap.parse_args()


MIXES = {"all": ((0, 0, 1, 0, 2), 200), "tp_pp": ((0, 0, 1, 0), 250), "dp": ((2,), 200)}   # op pattern (0 TP, 1 PP, 2 DP), repetitions


def workload(n_windows, rank=0, mix="all"):
    import tracegen as tg
    pattern, reps = MIXES[mix]
    spec = tg.cfg4(reps=reps, n_windows=n_windows, pattern=pattern)
    spec.seed += 1000 * rank
    return spec


def class_units(spec):
    """Records and groups per window, split by the kernel that reduces them (n <= 8, <= 128, <= 1024, larger)."""
    out = {"small": [0, 0], "warp": [0, 0], "mid": [0, 0], "large": [0, 0]}
    for f, fam in enumerate(spec.families):
        G, n = fam.members.shape
        ops = spec.pattern.count(f) * spec.reps
        k = "small" if n <= 8 else ("warp" if n <= 128 else ("mid" if n <= 1024 else "large"))
        out[k][0] += G * n * ops
        out[k][1] += G * ops
    return out


def peak_hbm():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return HBM_FALLBACK_GBS, "fallback"


def max_over_ranks(ms, device):
    """The slowest rank's elapsed time (all-reduce MAX over the default process group; identity for one rank)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.strip().splitlines():
            p = [x.strip() for x in line.split(",")]
            if len(p) < 8:
                continue
            try:
                sm.append(float(p[0])); mx.append(float(p[1]))
            except ValueError:
                continue
            for name, v in zip(names, p[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def time_oracle(spec, windows, gen_device="cpu"):
    """CPU oracle (single thread) on the given windows of the workload: records, seconds."""
    import oracle as orc
    import tracegen as tg
    o = orc.Oracle()
    for cid, ranks, seq0 in tg.registry(spec):
        o.comm_register(cid, ranks, seq0)
    n_rec, secs = 0, 0.0
    for w in windows:
        win = tg.gen_window(spec, w, device=gen_device)
        cols = {k: v.cpu().numpy() for k, v in win.cols.items()}
        t0 = time.perf_counter()
        o.upload(w, cols)
        o.analyze(w, 1, win.now_ns)
        o.sizes(w)
        secs += time.perf_counter() - t0
        n_rec += win.n_rec
        o.release(w)
    return n_rec, secs


def run_reference(args, rank):
    if rank != 0:
        return
    spec = workload(args.windows)
    n_rec = secs = 0
    for s in range(args.warmup + args.steps):
        r, t = time_oracle(spec, [s % spec.n_windows])
        if s >= args.warmup:
            n_rec += r; secs += t
    value = n_rec / secs
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": "cfg4 streaming slow mix: 4,096 ranks (TP8 x PP8 x DP64), windows of 1,000 ops per rank",
                   "records_per_step": n_rec // args.steps},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": "one window (4.096 M records) of the workload per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_ours(args, rank, world, local_rank):
    import torch
    import torch.distributed as dist
    import paper_2605_04478_b200 as ccld
    import tracegen as tg

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    cpu_base = None
    if rank == 0 and world == 1 and args.cpu_windows > 0:
        spec0 = workload(args.windows, 0, args.mix)
        r, t = time_oracle(spec0, list(range(min(args.cpu_windows, spec0.n_windows))), gen_device=dev)
        cpu_base = {"value": r / t, "unit": UNIT, "cores": 1, "kind": "oracle",
                    "sample": "%d of %d windows (%.3f M records), single thread" % (min(args.cpu_windows, spec0.n_windows), spec0.n_windows, r / 1e6)}

    spec = workload(args.windows, rank, args.mix)
    NW = spec.n_windows
    an = ccld.Analyzer(device=local_rank)
    for cid, ranks, seq0 in tg.registry(spec):
        an.comm_register(cid, ranks, 0, seq0)
    n_rec = 0
    now = 0
    for w in range(NW):
        win = tg.gen_window(spec, w, device=dev)
        an.trace_upload(w, win.cols)
        n_rec += win.n_rec
        now = win.now_ns
    torch.cuda.synchronize()

    def step():
        an.reset()
        an.analyze_window(0, NW, now)

    for _ in range(args.warmup):
        step()
    an.timing_enable(True)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local_rank)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1)
    kt = an.get_kernel_times()
    an.timing_enable(False)
    ms = max_over_ranks(ms, dev)
    value = world * n_rec * args.steps / (ms * 1e-3)

    # sanity: the injected ranks are the suspects
    v = an.get_verdict(NW - 1)
    sus = v["suspects"]
    found = {"stragglers": sorted(set(int(r) for r in sus["rank"][sus["kind"] == 1])),
             "slow_links": sorted(set(int(r) for r in sus["rank"][sus["kind"] == 2]))}
    recovered = found["stragglers"] == spec.truth["stragglers"] and found["slow_links"] == spec.truth["slow_links"]

    # ---- roofline of the dominant kernel ----
    units = class_units(spec)
    alg = {   # algorithmic bytes one launch moves (per window: records, groups of the class)
        "k_seq_range": lambda: NW * 8 * sum(u[0] for u in units.values()),
        "k_slot_scatter": lambda: NW * (12 + 4) * sum(u[0] for u in units.values()),
        "k_reduce_fused": lambda: NW * ((4 + 33 + 1) * (units["small"][0] + units["warp"][0]) + ROW_BYTES * (units["small"][1] + units["warp"][1])),
        "k_reduce_mid": lambda: NW * ((4 + 33 + 1) * units["mid"][0] + ROW_BYTES * units["mid"][1]),
        "k_reduce_large": lambda: NW * ((4 + 33 + 1) * units["large"][0] + ROW_BYTES * units["large"][1]),
    }
    dom = max(kt, key=lambda k: kt[k]["ms"])
    peak, peak_kind = peak_hbm()
    d_ms = kt[dom]["ms"] / max(kt[dom]["launches"], 1)
    d_bytes = alg.get(dom, lambda: 0)()
    achieved = d_bytes / (d_ms * 1e-3) / 1e9 if d_ms > 0 else 0.0
    path_bytes = REC_BYTES * n_rec + n_rec + ROW_BYTES * NW * sum(u[1] for u in units.values())
    path_gbs = path_bytes * args.steps / (ms * 1e-3) / 1e9
    tpr = NCU_TRAFFIC_PER_RECORD.get(dom)
    traffic = tpr * NW * (units["small"][0] + units["warp"][0]) if tpr is not None else None   # records of the kernel's classes
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic, "peak_source": peak_kind, "ms_per_launch": d_ms, "algorithmic_bytes_per_launch": d_bytes,
                "kernels_ms_per_step": {k: kt[k]["ms"] / args.steps for k in kt},
                "whole_path": {"algorithmic_bytes_per_step": path_bytes, "achieved": path_gbs, "frac": path_gbs / peak}}
    # every launch of the fused reduce kernel is followed by one of k_reduce_deferred (timed inside the same event pair)
    # and every launch of k_window_decide is preceded by one of k_window_rounds
    launches = sum(x["launches"] for x in kt.values()) + kt["k_reduce_fused"]["launches"] + kt["k_window_decide"]["launches"]

    # ---- end to end: host buffers -> upload -> analyse -> verdict ----
    NE = min(args.e2e_windows, NW)
    e2e = None
    if NE > 0:
        an_e = ccld.Analyzer(device=local_rank)
        for cid, ranks, seq0 in tg.registry(spec):
            an_e.comm_register(cid, ranks, 0, seq0)
        host, e_rec = [], 0
        for w in range(NE):
            win = tg.gen_window(spec, w, device=dev)
            host.append({k: t.cpu().pin_memory() for k, t in win.cols.items()})
            e_rec += win.n_rec
        del win
        h2d = sum(t.numel() * t.element_size() for cols in host for t in cols.values())
        d2h = 0

        def e2e_step():
            nonlocal d2h
            for w in range(NE):
                an_e.trace_upload(w, host[w])
            an_e.analyze_window(0, NE, now)
            vv = an_e.get_verdict(NE - 1)
            d2h = (NE * 8 * 8 + 16 * 8 + 104 * vv["n_comm_rows_total"] + 16 * min(vv["n_alerts_total"], 1024)
                   + 24 * vv["n_suspects_total"] + 4)
            for w in range(NE):
                an_e.window_release(w)
            an_e.reset()

        for _ in range(max(1, min(args.warmup, 3))):
            e2e_step()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e_steps = max(1, min(args.steps, 5))
        e0.record()
        for _ in range(e_steps):
            e2e_step()
        e1.record()
        torch.cuda.synchronize()
        e_ms = e0.elapsed_time(e1)
        e_ms = max_over_ranks(e_ms, dev)
        e2e = {"value": world * e_rec * e_steps / (e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "windows_per_step": NE, "steps": e_steps, "ms_per_step": e_ms / e_steps}
        an_e.close()

    # ---- counter changes per op from raw probe samples (the step before the path), timed on its own ----
    rates = None
    NR = min(args.rate_windows, NW)
    if NR > 0:
        win = tg.gen_window(spec, 0, device=dev)
        ticks = tg.gen_ticks(win.cols, spec.n_ranks)
        call = lambda: an.derive_rates(win.cols["rank"], win.cols["t_enter"], win.cols["t_exit"], ticks["tick_off"], ticks["tick_ns"],
                                       ticks["send_count"], ticks["recv_count"])
        for _ in range(3):
            call()
        torch.cuda.synchronize()
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        r0.record()
        for _ in range(NR * 5):
            call()
        r1.record()
        torch.cuda.synchronize()
        r_ms = r0.elapsed_time(r1) / (NR * 5)
        n_t = int(ticks["tick_ns"].numel())
        r_bytes = 16 * n_t + 28 * win.n_rec              # ticks read once (time, two counters); rank and times read, two counts written
        rates = {"records": win.n_rec, "ticks": n_t, "ms_per_window": r_ms, "algorithmic_bytes": r_bytes,
                 "achieved": r_bytes / (r_ms * 1e-3) / 1e9, "unit": "GB/s", "frac": r_bytes / (r_ms * 1e-3) / 1e9 / peak, "launches_per_window": 4}
        del win, ticks

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int64", "data": "synthetic",
            "config": {"workload": "cfg4 streaming slow mix: 4,096 ranks (TP8 x PP8 x DP64), %d windows of %s ops per rank, rank-major upload order%s"
                                   % (NW, format(spec.ops_per_window, ","), "" if args.mix == "all" else " (--mix %s: one communicator class only)" % args.mix),
                       "records_per_gpu": n_rec, "bytes_per_record": REC_BYTES, "l2": "inputs larger than L2 (%.1f GB of columns per GPU)" % (n_rec * REC_BYTES / 1e9),
                       "injected_ranks_recovered": recovered},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "cpu_baseline": cpu_base,
            "derive_rates": rates,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.gpus != world:
        if world == 1 and args.gpus > 1:
            sys.exit("for --gpus N > 1 launch with: python -m torch.distributed.run --nnodes=1 --nproc-per-node N "
                     "--master-addr 127.0.0.1 --master-port P bench.py --gpus N ...")
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
