"""Parity at full size, in the launch configuration the benchmark times.

All five configurations are analysed at their stated sizes somewhere in the GPU suite: the tiny slow case, the
512-rank job and the hang case in test_gpu_parity.py; the streaming slow mix, its one-communicator variant and the
16,384-rank scale stress here.

The streaming slow-mix workload (4,096 ranks, 100 windows of 1,000 ops per rank, 409.6 M records) is
generated on the GPU and analysed in ONE call, exactly as bench.py does. The oracle then recomputes
sampled windows one by one (each on a fresh oracle: the per-op table, flags, slot permutation and
counts do not depend on earlier windows), and the first two windows in sequence for the stateful
outputs. Properties that hold at any size are checked on every window.
"""
import os

import numpy as np
import pytest
import torch

import oracle as orc
import tracegen as tg
from parity import compare_window, same, close

pytestmark = pytest.mark.gpu


def test_cfg4_full_size_in_the_bench_configuration():
    import paper_2605_04478_b200 as ccld
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * 2**30:
        pytest.skip("needs about 30 GB of device memory")
    spec = tg.cfg4()
    NW = spec.n_windows
    assert NW == 100 and tg.records_per_window(spec) == 4_096_000
    an = ccld.Analyzer()
    reg = tg.registry(spec)
    for cid, ranks, seq0 in reg:
        an.comm_register(cid, ranks, 0, seq0)
    sample = [0, 1, 37, 99]
    kept = {}
    for w in range(NW):
        win = tg.gen_window(spec, w, device="cuda")
        an.trace_upload(w, win.cols)
        if w in sample:
            kept[w] = {k: v.cpu() for k, v in win.cols.items()}
        now = win.now_ns
    an.analyze_window(0, NW, now)

    # properties on every window
    tot_flags = 0
    for w in range(NW):
        v = an.get_verdict(w)
        assert v["n_records"] == 4_096_000 and v["n_groups"] == 422_400 and v["n_slots"] == 4_096_000
        assert v["n_complete"] == 422_400 and v["n_incomplete"] == 0 and v["n_rejected"] == 0 and v["error_bits"] == 0
        assert v["n_analysed"] == 422_400 and v["n_comm_rows_total"] == 1088 and v["n_alerts_total"] == 0
        tot_flags += v["n_flag_skew"] + v["n_flag_dur"]
    st = an.get_rank_stats(spec.n_ranks)
    assert int(st["votes"].sum()) == tot_flags                       # vote total = flag total
    assert (st["ops"] == 100_000).all() and (st["bw_cnt"] == 100_000).all()
    sus = v["suspects"]
    assert sorted(set(int(r) for r in sus["rank"][sus["kind"] == 1])) == spec.truth["stragglers"]
    assert sorted(set(int(r) for r in sus["rank"][sus["kind"] == 2])) == spec.truth["slow_links"]

    # sampled windows against the oracle, element by element (stateless outputs)
    for w in sample[2:]:
        o = orc.Oracle()
        for cid, ranks, seq0 in reg:
            o.comm_register(cid, ranks, seq0)
        o.upload(w, kept[w]); o.analyze(w, 1, now)
        compare_window(an, o, w, stateless_only=True)
        t = an.get_optable(w)
        assert (t["arrival_skew"] >= 0).all() and (t["t_min"] <= t["med_dur"]).all() and (t["med_dur"] <= t["t_max"]).all()
    # the first two windows in sequence: communicator rows and cumulative state too
    o = orc.Oracle()
    for cid, ranks, seq0 in reg:
        o.comm_register(cid, ranks, seq0)
    for w in (0, 1):
        o.upload(w, kept[w])
    o.analyze(0, 2, now)
    for w in (0, 1):
        compare_window(an, o, w)
    # per-rank votes after two windows: analyse the same two windows alone on a second context
    an2 = ccld.Analyzer()
    for cid, ranks, seq0 in reg:
        an2.comm_register(cid, ranks, 0, seq0)
    for w in (0, 1):
        an2.trace_upload(w, {k: v.cuda() for k, v in kept[w].items()})
    an2.analyze_window(0, 2, now)
    a, b = an2.get_rank_stats(spec.n_ranks), o.rank_stats(spec.n_ranks)
    for k in ("votes", "ops", "bw_cnt"):
        same(a[k], b[k], k)
    close(a["bw_sum"], b["bw_sum"], "bw_sum")
    an2.close()
    del o, kept
    # votes, op counts and bandwidth sums add up over windows: the oracle analyses each of the 100 windows on its own
    # (several host cores side by side), and the sums and the suspect list they give must be the library's after 100 windows
    cumulative_against_independent_oracles(an, spec, reg, NW, now)


def cumulative_against_independent_oracles(an, spec, reg, n_windows, now, v_last=None):
    threads = max(1, min(16, os.cpu_count() or 1))

    def windows():
        for w in range(n_windows):
            win = tg.gen_window(spec, w, device="cuda")
            yield w, {k: v.cpu().numpy() for k, v in win.cols.items()}, now

    tot, sizes, n_rec = orc.analyze_windows_independently(reg, windows(), spec.n_ranks, threads=threads)
    st = an.get_rank_stats(spec.n_ranks)
    for k in ("votes", "ops", "bw_cnt"):
        same(st[k], tot[k], "cumulative " + k)
    close(st["bw_sum"], tot["bw_sum"], "cumulative bw_sum")
    for w in range(n_windows):
        v = an.get_verdict(w, check=False)
        for k in ("n_records", "n_groups", "n_complete", "n_incomplete", "n_analysed", "n_flag_skew", "n_flag_dur", "n_barrier"):
            assert v[k] == sizes[w][k], (w, k, v[k], sizes[w][k])
    merged = orc.Oracle()
    merged.add_rank_stats(tot)
    sa, sb = an.get_verdict(n_windows - 1, check=False)["suspects"], merged.suspects()
    for k in ("kind", "rank", "votes", "ops"):
        same(sa[k], sb[k], "suspect " + k)
    close(sa["mean_busbw"], sb["mean_busbw"], "suspect mean_busbw")


def fresh_oracle(reg):
    o = orc.Oracle()
    for cid, ranks, seq0 in reg:
        o.comm_register(cid, ranks, seq0)
    return o


def test_cfg4w_full_size_one_4096_rank_communicator():
    """The streaming workload read as ONE 4,096-rank communicator: 100 windows of 1,000 AllReduces, 409.6 M records,
    analysed in one call. Every group goes through the radix-select kernel."""
    import paper_2605_04478_b200 as ccld
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * 2**30:
        pytest.skip("needs about 30 GB of device memory")
    spec = tg.cfg4w()
    NW = spec.n_windows
    assert NW == 100 and tg.records_per_window(spec) == 4_096_000 and spec.families[0].members.shape == (1, 4096)
    an = ccld.Analyzer()
    reg = tg.registry(spec)
    for cid, ranks, seq0 in reg:
        an.comm_register(cid, ranks, 0, seq0)
    sample = [0, 1, 58, 99]
    kept = {}
    for w in range(NW):
        win = tg.gen_window(spec, w, device="cuda")
        an.trace_upload(w, win.cols)
        if w in sample:
            kept[w] = {k: v.cpu() for k, v in win.cols.items()}
        now = win.now_ns
    an.analyze_window(0, NW, now)
    tot_flags = 0
    for w in range(NW):
        v = an.get_verdict(w)
        assert v["n_records"] == 4_096_000 and v["n_groups"] == 1000 and v["n_slots"] == 4_096_000
        assert v["n_complete"] == 1000 and v["n_analysed"] == 1000 and v["n_rejected"] == 0 and v["error_bits"] == 0
        assert v["n_comm_rows_total"] == 1 and v["n_alerts_total"] == 0
        tot_flags += v["n_flag_skew"] + v["n_flag_dur"]
    st = an.get_rank_stats(spec.n_ranks)
    assert int(st["votes"].sum()) == tot_flags and (st["ops"] == 100_000).all() and (st["bw_cnt"] == 100_000).all()
    sus = v["suspects"]
    assert sorted(set(int(r) for r in sus["rank"][sus["kind"] == 1])) == spec.truth["stragglers"]
    assert sorted(set(int(r) for r in sus["rank"][sus["kind"] == 2])) == spec.truth["slow_links"]
    for w in sample[2:]:
        o = fresh_oracle(reg)
        o.upload(w, kept[w]); o.analyze(w, 1, now)
        compare_window(an, o, w, stateless_only=True)
    o = fresh_oracle(reg)
    for w in (0, 1):
        o.upload(w, kept[w])
    o.analyze(0, 2, now)
    for w in (0, 1):
        compare_window(an, o, w)


def test_cfg5_full_size_16384_ranks_with_concurrent_hang():
    """Scale stress at its stated size: 16,384 ranks, 50 windows, 819 M records (36.9 GB of columns) generated on the
    device and analysed in one call; groups of 8, 128 and 2,048 ranks plus the 1,024-rank ring that hangs at step 41 in
    window 25. Sampled windows (the first, the hang window, the last) against the oracle element by element; counts on
    every window; all 32 injected ranks and the ring's root recovered."""
    import paper_2605_04478_b200 as ccld
    free, _ = torch.cuda.mem_get_info()
    if free < 80 * 2**30:
        pytest.skip("needs about 60 GB of device memory")
    spec = tg.cfg5()
    NW, HW = spec.n_windows, spec.hang.window
    assert NW == 50 and HW == 25 and spec.n_ranks == 16_384
    an = ccld.Analyzer()
    reg = tg.registry(spec)
    for cid, ranks, seq0 in reg:
        an.comm_register(cid, ranks, 0, seq0)
    sample = [0, HW, NW - 1]
    kept, n_rec = {}, []
    for w in range(NW):
        win = tg.gen_window(spec, w, device="cuda")
        an.trace_upload(w, win.cols, win.frames, win.n_channels)
        if w in sample:
            kept[w] = ({k: v.cpu() for k, v in win.cols.items()}, None if win.frames is None else {k: v.cpu() for k, v in win.frames.items()}, win.n_channels)
        n_rec.append(win.n_rec)
        now = win.now_ns
    del win
    assert sum(n_rec) > 819_000_000
    an.analyze_window(0, NW, now)
    # per window: 16,384 ranks x 1,000 ops in groups of 8 / 128 / 2,048 plus ten ops of the 1,024-rank ring until it hangs
    n_groups = 2048 * 500 + 128 * 250 + 8 * 250
    alerts, tot_flags = [], 0
    for w in range(NW):
        v = an.get_verdict(w)
        ring_ops = 10 if w < HW else (6 if w == HW else 0)          # the hung op is the sixth of its window
        assert v["n_records"] == n_rec[w] == 16_384_000 + 1024 * ring_ops, (w, v["n_records"])
        assert v["n_groups"] == n_groups + ring_ops and v["n_rejected"] == 0 and v["error_bits"] == 0
        assert v["n_incomplete"] == (1 if w == HW else 0) and v["n_complete"] == v["n_groups"] - v["n_incomplete"]
        assert v["n_analysed"] == v["n_complete"]
        tot_flags += v["n_flag_skew"] + v["n_flag_dur"]
        alerts += [(w, int(c), int(s)) for c, s in zip(v["alerts"]["comm"], v["alerts"]["seq"])]
    st = an.get_rank_stats(spec.n_ranks)
    assert int(st["votes"].sum()) == tot_flags
    ring_fam = spec.families[3]
    assert alerts == [(HW, ring_fam.comm_id0, spec.hang.seq)]
    sus = v["suspects"]
    assert sorted(set(int(r) for r in sus["rank"][sus["kind"] == 1])) == spec.truth["stragglers"]
    assert sorted(set(int(r) for r in sus["rank"][sus["kind"] == 2])) == spec.truth["slow_links"]
    # sampled windows element by element; window 0 also with its communicator rows (no earlier state to carry)
    for w in sample:
        o = fresh_oracle(reg)
        cols, frames, nch = kept[w]
        o.upload(w, cols, frames, nch); o.analyze(w, 1, now)
        compare_window(an, o, w, stateless_only=(w != 0))
        if w == HW:
            from parity import compare_hang
            h = compare_hang(an, o, w, ring_fam.comm_id0, spec.hang.seq)
            assert h["cls"] == 3 and list(h["roots"]) == spec.truth["hang_root"] and h["stuck_step"] == 41
        del o


def test_derive_rates_full_window_in_the_bench_configuration():
    """One cfg4 window with its raw probe samples (4.1 M records, 21 M ticks), derived in one call as bench.py does.
    The oracle recomputes a sample of the records (it walks every tick of a record's rank); properties that hold at any
    size are checked on all of them."""
    import paper_2605_04478_b200 as ccld
    spec = tg.cfg4(n_windows=1)
    win = tg.gen_window(spec, 0, device="cuda")
    ticks = tg.gen_ticks(win.cols, spec.n_ranks)
    an = ccld.Analyzer()
    s, r = an.derive_rates(win.cols["rank"], win.cols["t_enter"], win.cols["t_exit"], ticks["tick_off"], ticks["tick_ns"],
                           ticks["send_count"], ticks["recv_count"])
    torch.cuda.synchronize()
    n = win.n_rec
    assert n == 4_096_000 and int(ticks["tick_ns"].numel()) > 20_000_000
    s = s.cpu().numpy().view(np.uint32); r = r.cpu().numpy().view(np.uint32)
    c = {k: v.cpu().numpy() for k, v in win.cols.items() if k in ("rank", "t_enter", "t_exit")}
    k = {k: v.cpu().numpy() for k, v in ticks.items()}
    # sampled records, spread over every rank and the whole window, plus the first and last of the upload
    rng = np.random.default_rng(7)
    pick = np.unique(np.concatenate([rng.integers(0, n, 6000), np.arange(0, 64), np.arange(n - 64, n)]))
    es, er = orc.derive_rates(c["rank"][pick], c["t_enter"][pick], c["t_exit"][pick], k["tick_off"], k["tick_ns"], k["send_count"], k["recv_count"])
    same(s[pick], es, "send_chg"); same(r[pick], er, "recv_chg")
    # a count never exceeds the ticks inside the op, and an op of this trace (8 sends spread over its duration) that
    # covers at least one tick shows at least one change of the counter that rounds up
    per = (c["t_exit"] - c["t_enter"]) // 1_000_000 + 1
    assert (s <= per).all() and (r <= per).all()
    assert (r[per >= 3] >= 1).all()
    # the same call again gives the same columns (the scratch block is reused)
    s2, r2 = an.derive_rates(win.cols["rank"], win.cols["t_enter"], win.cols["t_exit"], ticks["tick_off"], ticks["tick_ns"],
                             ticks["send_count"], ticks["recv_count"])
    torch.cuda.synchronize()
    assert np.array_equal(s2.cpu().numpy().view(np.uint32), s) and np.array_equal(r2.cpu().numpy().view(np.uint32), r)
