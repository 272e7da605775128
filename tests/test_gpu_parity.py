"""Parity of the CUDA library with the CPU oracle, through the C ABI, on the same seeded inputs.

Integer quantities (skews, durations, medians, MADs, flags, votes, roots) must be identical;
fp64 bandwidths, R and P within 1e-9 relative.
"""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2605_04478_b200 as ccld
import tracegen as tg
from helpers import ALLGATHER, MiB, frames_from, group_trace, make_cols
from parity import compare_cumulative, compare_hang, compare_window, make_pair

pytestmark = pytest.mark.gpu


def run_spec(spec, windows=None, order="rank_major", batch=True, device="cpu", params=None):
    """Uploads the given windows of `spec` to both sides, analyses them and compares everything."""
    reg = tg.registry(spec)
    an, o = make_pair(reg, params)
    windows = list(range(spec.n_windows)) if windows is None else windows
    wins = []
    for w in windows:
        win = tg.gen_window(spec, w, device=device, order=order)
        wins.append(win)
        an.trace_upload(w, win.cols, win.frames, win.n_channels)
        assert o.upload(w, win.cols, win.frames, win.n_channels) == 0
    now = wins[-1].now_ns
    if batch:
        an.analyze_window(windows[0], len(windows), now)
    else:
        for w in windows:
            an.analyze_window(w, 1, now)
    assert o.analyze(windows[0], len(windows), now) == 0
    verdicts = [compare_window(an, o, w)[0] for w in windows]
    sus = compare_cumulative(an, o, spec.n_ranks, windows[-1])
    return an, o, verdicts, sus


# ---------------------------------------------------------------- the benchmark configurations
def test_cfg1_tiny_slow_case():
    spec = tg.cfg1()
    an, o, v, sus = run_spec(spec)
    assert v[0]["n_records"] == 8000 and v[0]["n_groups"] == 1000
    assert sorted(set(sus["rank"])) == [5] and list(sus["kind"]) == [1]


def test_cfg2_full_size_512_ranks():
    spec = tg.cfg2()
    an, o, v, sus = run_spec(spec)
    assert sum(x["n_records"] for x in v) == 15_360_000
    assert sorted(set(int(r) for r in sus["rank"][sus["kind"] == 1])) == spec.truth["stragglers"]
    assert sorted(set(int(r) for r in sus["rank"][sus["kind"] == 2])) == spec.truth["slow_links"]


@pytest.mark.parametrize("order", ["arrival", "shuffled"])
def test_cfg2_other_upload_orders(order):
    spec = tg.cfg2(reps=100, n_windows=2)
    run_spec(spec, order=order, batch=False)


def test_cfg3_hang_case():
    spec = tg.cfg3()
    an, o, v, sus = run_spec(spec)
    a = v[0]["alerts"]
    assert list(a["comm"]) == [7] and list(a["seq"]) == [100]
    h = compare_hang(an, o, 0, 7, 100)
    assert h["cls"] == 3 and list(h["roots"]) == [1793] and h["stuck_step"] == 23
    compare_hang(an, o, 0, 3, 100)       # a ring that completed
    compare_hang(an, o, 0, 7, 101)       # an op nobody entered
    compare_hang(an, o, 0, 7, 50)


def test_cfg4_scaled_three_windows_device_resident():
    # same structure as the streaming configuration (4,096 ranks, TP8 x PP8 x DP64), 100 ops per rank and window,
    # generated on the GPU and borrowed by the library
    spec = tg.cfg4(reps=20, n_windows=3)
    an, o, v, sus = run_spec(spec, device="cuda")
    assert v[0]["n_records"] == 409_600
    assert sorted(set(int(r) for r in sus["rank"][sus["kind"] == 1])) == spec.truth["stragglers"]
    assert sorted(set(int(r) for r in sus["rank"][sus["kind"] == 2])) == spec.truth["slow_links"]


def test_cfg4w_one_4096_rank_communicator():
    spec = tg.cfg4w(reps=21, n_windows=2)
    an, o, v, sus = run_spec(spec)
    assert v[0]["n_groups"] == 21 and v[0]["n_analysed"] == 21


def test_cfg5_scaled_16384_ranks_with_hang():
    # full rank count (groups of 8, 128, 2,048 and the hung 1,024-rank ring), one pattern repetition per window
    spec = tg.cfg5(reps=1, n_windows=3, hang_window=1)
    an, o, v, sus = run_spec(spec)
    alerts = [(w, int(c), int(s)) for w, x in enumerate(v) for c, s in zip(x["alerts"]["comm"], x["alerts"]["seq"])]
    assert len(alerts) == 1
    w, c, s = alerts[0]
    h = compare_hang(an, o, w, c, s)
    assert h["cls"] == 3 and list(h["roots"]) == spec.truth["hang_root"] and h["stuck_step"] == 41


# ---------------------------------------------------------------- group sizes across the three kernels
def sized_spec(sizes, reps, seed=11, ties=False):
    fams, r0, cid = [], 0, 0
    for n in sizes:
        m = torch.arange(r0, r0 + 2 * n, dtype=torch.int64).reshape(2, n)
        m[1] = m[1].flip(0)                                  # ring order differs from rank order
        fams.append(tg.Family(f"n{n}", m, (tg.OP_ALLREDUCE, tg.OP_ALLGATHER), cid,
                              bytes_choices=(MiB,) if ties else None))
        r0 += 2 * n; cid += 2
    s = tg.Spec("sized", seed, r0, fams, list(range(len(sizes))), reps, 2)
    s.faults = [tg.Fault(3, "delay_exp", 300, 400_000), tg.Fault(r0 - 2, "bw", factor_milli=500)]
    if ties:
        s.jitter_ns = 3                                       # enter times collide: many equal skews
    return s


@pytest.mark.parametrize("sizes,reps", [
    ((1, 2, 3, 4, 5, 6, 7, 8), 300),                          # thread-per-group kernel, ragged tiles
    ((9, 15, 16, 17, 31, 32, 33), 150),                       # bitonic kernel, small paddings
    ((63, 64, 65, 100, 128, 255, 256, 257), 37),
    ((511, 512, 1000, 1023, 1024), 5),
    ((1025, 2048, 3000, 4096), 9),                            # radix-select kernel, tiles of 8 groups + tail
    ((8192,), 3),                                             # the largest communicator the library takes
])
def test_group_sizes(sizes, reps):
    run_spec(sized_spec(sizes, reps))


def test_group_sizes_with_many_ties():
    run_spec(sized_spec((4, 8, 24, 64, 200, 1500), 20, ties=True))


def test_wide_value_ranges_and_damaged_groups_in_every_class():
    """Skews and durations more than 2^32 ns apart (64-bit keys), and missing / in-flight / mismatched / barrier
    groups, for group sizes of every kernel and every lanes-per-group layout."""
    rng = np.random.default_rng(5)
    recs, comms, r0 = [], [], 0
    for cid, n in enumerate((5, 8, 12, 24, 40, 64, 100, 128, 200, 1100)):
        ranks = list(range(r0, r0 + n)); r0 += n
        comms.append((cid, ranks, 0))
        n_seq = 70 if n <= 128 else 6
        durs = rng.integers(1_000_000, 1_200_000, size=(n_seq, n)).tolist()
        ents = rng.integers(0, 40_000, size=(n_seq, n)).tolist()
        durs[1][n // 2] = 7_000_000_000                       # duration spread above 2^32 ns
        ents[2][n - 1] = 5_000_000_000                        # skew spread above 2^32 ns
        durs[3][0] = 6_000_000_000; ents[3][n // 3] = 4_400_000_000
        durs[n_seq - 1][n - 1] = 2**33                        # in the last (ragged) tile
        g = group_trace(durs, ents, comm=cid, ranks=ranks, spacing=10_000_000_000, bytes=MiB)
        by_key = {(r["seq"], r["rank"]): r for r in g}
        del by_key[(4, ranks[n - 1])]                         # missing member
        by_key[(5, ranks[1])]["t_exit"] = -1                  # in flight
        by_key[(n_seq - 2, ranks[n // 2])]["bytes"] = 2 * MiB  # op-set mismatch
        for r in g:
            if r["seq"] == 0: r["bytes"] = 3                  # barrier
        recs += list(by_key.values())
    hand_pair(recs, comms, now=10**13)


# ---------------------------------------------------------------- edge cases
def hand_pair(recs, comms, params=None, now=10**12, with_rates=True, frames=None, n_channels=0, expect_rc=0):
    an, o = make_pair(comms, params)
    cols = make_cols(recs, with_rates)
    an.trace_upload(0, cols, frames, n_channels)
    assert o.upload(0, cols, frames, n_channels) == 0
    an.analyze_window(0, 1, now)
    assert o.analyze(0, 1, now) == 0
    compare_window(an, o, 0, expect_rc=expect_rc)
    return an, o


def test_rejected_records_and_incomplete_groups():
    recs = group_trace([[5, 5, 5, 5], [5, 5, 5, 5], [5, 5, 5, 5]], seq0=10)
    recs = [r for r in recs if not (r["seq"] == 11 and r["rank"] == 2)]
    recs.append(dict(rank=0, comm=99, seq=10, t_enter=1, t_exit=2))
    recs.append(dict(rank=77, comm=0, seq=10, t_enter=1, t_exit=2))
    recs.append(dict(rank=77, comm=0, seq=14, t_enter=1, t_exit=2))      # non-member widens the op-counter range
    recs.append(dict(rank=1, comm=0, seq=3, t_enter=1, t_exit=2))
    hand_pair(recs, [(0, [0, 1, 2, 3], 10)], expect_rc=-4)
    hand_pair(recs[:-4] + recs[-3:], [(0, [0, 1, 2, 3], 10)], expect_rc=-5)
    hand_pair(recs[:-4] + recs[-1:], [(0, [0, 1, 2, 3], 10)], expect_rc=-6)


def test_barrier_small_group_mismatch_bad_times_no_rates():
    recs = group_trace([[5, 5, 5, 900]], comm=0, bytes=3)
    recs += group_trace([[5, 5, 5, 900]], comm=1, ranks=[4, 5, 6, 7], bytes=4)
    recs += group_trace([[5, 5, 900]], comm=2, ranks=[8, 9, 10])
    recs += group_trace([[5, 5, 5, 900]], comm=3, ranks=[12, 13, 14, 15], op=ALLGATHER, bytes=3)
    mism = group_trace([[5, 6, 7, 8]] * 2, comm=4, ranks=[16, 17, 18, 19])
    mism[5]["bytes"] = 8 * MiB
    bad = group_trace([[5, 6, 7, 8]] * 2, comm=5, ranks=[20, 21, 22, 23])
    bad[1]["t_exit"] = bad[1]["t_enter"] - 3
    bad[6]["t_enter"] = -5
    comms = [(0, [0, 1, 2, 3], 0), (1, [4, 5, 6, 7], 0), (2, [8, 9, 10], 0), (3, [12, 13, 14, 15], 0),
             (4, [16, 17, 18, 19], 0), (5, [20, 21, 22, 23], 0), (6, [30, 31], 0)]
    hand_pair(recs + mism + bad, comms)
    hand_pair(recs + mism + bad, comms, with_rates=False)


def test_slow_location_classes_and_repetition():
    MS = 1_000_000
    comms = [(0, [0, 1, 2, 3], 0)]

    def coupled(enter_off, own, chg, seq):
        last = max(enter_off)
        return [dict(rank=i, comm=0, seq=seq, t_enter=10**9 * (seq + 1) + e, t_exit=10**9 * (seq + 1) + last + d, send_chg=c, recv_chg=1)
                for i, (e, d, c) in enumerate(zip(enter_off, own, chg))]
    wins = [coupled([0, 0, 20 * MS, 0], [2 * MS] * 4, [1] * 4, 0), coupled([0] * 4, [10 * MS] * 4, [2, 2, 2, 7], 1),
            coupled([0, 8 * MS, 0, 0], [10 * MS] * 4, [9, 2, 2, 2], 2), coupled([0] * 4, [2 * MS] * 4, [1] * 4, 3)]
    an, o = make_pair(comms, dict(tbase_init_ns=2 * MS))
    for w, r in enumerate(wins):
        cols = make_cols(r)
        an.trace_upload(w, cols); o.upload(w, cols)
    an.analyze_window(0, 2, 10**12); an.analyze_window(2, 2, 10**12)
    o.analyze(0, 4, 10**12)
    rows = [compare_window(an, o, w)[0]["comm_rows"] for w in range(4)]
    assert [int(r["cls"][0]) for r in rows] == [1, 2, 3, 0]
    assert [int(r["located"][0]) for r in rows] == [0, 1, 1, 0]


def test_baseline_becomes_dynamic_across_batches():
    durs = [[1000 + 10 * s + i for i in range(4)] for s in range(260)]
    durs[250][2] = 90_000
    recs = group_trace(durs)
    an, o = make_pair([(0, [0, 1, 2, 3], 0)], dict(tbase_init_ns=500))
    for w in range(4):
        cols = make_cols(recs[w * 260:(w + 1) * 260])
        an.trace_upload(w, cols); o.upload(w, cols)
    an.analyze_window(0, 1, 10**12); an.analyze_window(1, 3, 10**12)
    o.analyze(0, 4, 10**12)
    rows = [compare_window(an, o, w)[0]["comm_rows"] for w in range(4)]
    assert [int(r["baseline_static"][0]) for r in rows] == [1, 0, 0, 0] and int(rows[3]["m"][0]) == 100


def hang_records(n, seq, entered, done, ranks):
    recs = []
    for s in range(seq):
        recs += [dict(rank=ranks[i], comm=0, seq=s, t_enter=1000 + s, t_exit=2000 + s) for i in range(n)]
    for i in range(n):
        if i in entered:
            recs.append(dict(rank=ranks[i], comm=0, seq=seq, t_enter=10**9, t_exit=(10**9 + 5 if i in done else -1)))
    return recs


def test_hang_tree_leaves_and_tie_breaks():
    n, C = 6, 2
    ranks = [10, 11, 12, 13, 14, 15]
    comms = [(0, ranks, 0)]
    an, o = hand_pair(hang_records(n, 3, {0, 1, 2, 4}, set(), ranks), comms)
    assert compare_hang(an, o, 0, 0, 3)["cls"] == 1
    an, o = hand_pair(hang_records(n, 3, set(range(n)), {2}, ranks), comms)
    assert compare_hang(an, o, 0, 0, 3)["cls"] == 2
    recs = hang_records(n, 3, set(range(n)), set(), ranks)
    tot = {5: 4, 0: 4, 1: 4}
    cases = [
        [(ranks[i], 0, 3, [(9, 9), (9, 8)] if i != 4 else [(9, 7), (8, 6)]) for i in range(n)],
        [(ranks[i], 0, 3, [(tot.get(i, 6), tot.get(i, 6))] * C) for i in range(n)],
        [(ranks[i], 0, 3, [(5, 5)] * C) for i in range(n)],
        [(ranks[i], 0, 3, [(5, 5)] * C) for i in range(n) if i != 2],
        [(ranks[i], 0, 3, [(5, 5)] * C) for i in range(n)] + [(ranks[1], 0, 3, [(1, 1)] * C), (99, 0, 3, [(0, 0)] * C), (ranks[0], 0, 2, [(0, 0)] * C)],
    ]
    for entries in cases:
        an, o = hand_pair(recs, comms, frames=frames_from(entries, C), n_channels=C, now=10**9 + 400 * 10**9)
        assert compare_hang(an, o, 0, 0, 3)["cls"] == 3
    an, o = hand_pair(recs, comms)          # no frames at all
    compare_hang(an, o, 0, 0, 3)


def test_empty_window_capacity_and_call_order():
    import paper_2605_04478_b200 as ccld
    comms = [(0, [0, 1, 2, 3], 0), (1, [4, 5, 6, 7], 0)]
    an, o = make_pair(comms)
    empty = make_cols([])
    an.trace_upload(0, empty); o.upload(0, empty)
    cols = make_cols(group_trace([[5, 6, 7, 8]] * 3))
    an.trace_upload(1, cols); o.upload(1, cols)
    an.analyze_window(0, 2, 10**12); o.analyze(0, 2, 10**12)
    compare_window(an, o, 0); compare_window(an, o, 1)
    with pytest.raises(ccld.CcldError) as e:
        an.analyze_window(1, 1, 10**12)
    assert e.value.code == -9
    with pytest.raises(ccld.CcldError) as e:
        an.comm_register(5, [1, 2], 0, 0)
    assert e.value.code == -9
    with pytest.raises(ccld.CcldError) as e:
        an.get_verdict(7)
    assert e.value.code == -7
    with pytest.raises(ccld.CcldError) as e:
        an.analyze_window(0, 65536, 10**12)                  # more windows than one batch takes
    assert e.value.code == -8
    # op counters 0 and 4,000,000,000 in one window: the slot space would be absurd, the window is refused
    far = group_trace([[5, 6, 7, 8]]) + group_trace([[5, 6, 7, 8]], seq0=4_000_000_000)
    an.trace_upload(2, make_cols(far))
    an.analyze_window(2, 1, 10**12)
    v = an.get_verdict(2, check=False)
    assert v["rc"] == -8 and v["error_bits"] == 16 and v["n_groups"] == 0
    # the context still works afterwards
    an.reset()
    an.analyze_window(1, 1, 10**12)
    assert an.get_verdict(1)["n_complete"] == 3
    an2 = ccld.Analyzer()
    with pytest.raises(ccld.CcldError) as e:
        an2.comm_register(0, list(range(8193)))
    assert e.value.code == -8


def test_duplicate_record_is_reported():
    recs = group_trace([[5, 6, 7, 8]] * 2)
    recs.append(dict(recs[2]))
    an, o = make_pair([(0, [0, 1, 2, 3], 0)])
    an.trace_upload(0, make_cols(recs))
    an.analyze_window(0, 1, 10**12)
    v = an.get_verdict(0, check=False)
    assert v["rc"] == -10 and v["error_bits"] & 8 and v["n_rejected"] == 1


def test_reset_reproduces_the_same_results():
    spec = tg.cfg2(reps=50, n_windows=2)
    an, o, v, sus = run_spec(spec)
    an.reset()
    an.analyze_window(0, 2, 10**12)
    for w in range(2):
        compare_window(an, o, w)
    compare_cumulative(an, o, spec.n_ranks, 1)


def test_hang_sweep_locates_every_alert_in_one_launch():
    """Several hung communicators of different sizes, one per leaf of the decision tree (plus ties and missing frames):
    ccld_locate_hangs returns, alert by alert, what the oracle and ccld_locate_hang return."""
    C_ = 2
    recs, comms, entries, r0 = [], [], [], 0
    plan = [(6, "h1"), (40, "h3"), (8, "h2"), (130, "h3"), (5, "ok"), (12, "h3tie"), (9, "h1")]
    for cid, (n, kind) in enumerate(plan):
        ranks = list(range(r0, r0 + n)); r0 += n
        comms.append((cid + 3, ranks, 0))
        entered = set(range(n)) - ({1, n - 1} if kind == "h1" else set())
        done = {2, 3} if kind == "h2" else (set(range(n)) if kind == "ok" else set())
        for r in hang_records(n, 2 + cid, entered, done, ranks):
            r["comm"] = cid + 3
            recs.append(r)
        if kind.startswith("h3"):
            for i in range(n):
                if kind == "h3" and i == n // 2: continue                      # a member without a frame counts as zero
                v = 4 if (kind == "h3tie" and i in (3, 4, 5)) else 7
                entries.append((ranks[i], cid + 3, 2 + cid, [(v, v - 1)] * C_))
    an, o = hand_pair(recs, comms, frames=frames_from(entries, C_), n_channels=C_, now=10**9 + 400 * 10**9)
    al = an.get_verdict(0)["alerts"]
    assert len(al["comm"]) == 6                                                # every communicator but the completed one
    sweep = an.locate_hangs(0, cap=16, roots_stride=256)
    assert [(d["comm"], d["seq"]) for d in sweep] == list(zip(al["comm"].tolist(), al["seq"].tolist()))
    for d in sweep:
        b = o.locate_hang(0, d["comm"], d["seq"])
        assert d["cls"] == b["cls"] and d["n_roots_total"] == b["n_roots"], (d, b)
        for k in ("n_not_entered", "n_hung", "n_not_hung", "n_missing_frames", "stuck_step", "n_members", "min_total"):
            assert d[k] == b[k], (k, d[k], b[k])
        assert np.array_equal(d["roots"], b["roots"])
        a = an.locate_hang(0, d["comm"], d["seq"])
        assert a["cls"] == d["cls"] and np.array_equal(a["roots"], d["roots"])
    assert sorted(d["cls"] for d in sweep) == [1, 1, 2, 3, 3, 3]
    # truncation: fewer verdicts than alerts, short root lists
    few = an.locate_hangs(0, cap=2, roots_stride=1)
    assert len(few) == 2 and all(len(d["roots"]) <= 1 for d in few) and few[0]["n_roots_total"] == sweep[0]["n_roots_total"]


def test_state_export_import_continues_on_another_context():
    """Two windows on one analyzer, its state exported and imported into a fresh one, two more windows there: the second
    analyzer's windows, cumulative votes and suspects equal an oracle that saw all four windows in one life."""
    spec = tg.cfg2(reps=30, n_windows=4, tp=8, pp=2, dp=4)
    an_a, an_b, o = ccld.Analyzer(), ccld.Analyzer(), orc.Oracle()
    for cid, ranks, seq0 in tg.registry(spec):
        an_a.comm_register(cid, ranks, 0, seq0); an_b.comm_register(cid, ranks, 0, seq0); o.comm_register(cid, ranks, seq0)
    wins = [tg.gen_window(spec, w, device="cuda") for w in range(4)]
    for w in range(4):
        (an_a if w < 2 else an_b).trace_upload(w, wins[w].cols)
        o.upload(w, wins[w].cols)
    now = wins[-1].now_ns
    an_a.analyze_window(0, 2, now)
    blob = an_a.state_export()
    an_b.state_import(blob)
    an_b.analyze_window(2, 2, now)
    o.analyze(0, 4, now)
    for w in (0, 1):
        compare_window(an_a, o, w)
    for w in (2, 3):
        compare_window(an_b, o, w)
    compare_cumulative(an_b, o, spec.n_ranks, 3)
    assert an_b.state_export() != blob
    # a blob of another set of communicators is refused
    an_c = ccld.Analyzer()
    an_c.comm_register(0, [0, 1, 2, 3], 0, 0)
    with pytest.raises(ccld.CcldError):
        an_c.state_import(blob)
    with pytest.raises(ccld.CcldError):
        an_b.state_import(blob[:-8])


def test_opset_consistency_against_the_oracle():
    """Majority Operation Type Set and deviating ranks for groups of every kernel class, with and without the algorithm /
    protocol columns, with missing members, ties, an op nobody reported and an op outside the window's range."""
    rng = np.random.default_rng(41)
    recs, comms, r0 = [], [], 0
    for cid, n in enumerate((6, 40, 130, 1100)):
        ranks = list(range(r0, r0 + n)); r0 += n
        comms.append((cid, ranks, 0))
        g = group_trace([[5] * n] * 5, comm=cid, ranks=ranks)
        for x in g:
            if x["seq"] >= 1:
                x["op"] = int(rng.choice([0, 0, 0, 1])); x["bytes"] = int(rng.choice([4, 4, 4, 8])) * MiB
        if cid == 0:
            for x in g:
                if x["seq"] == 4: x["bytes"] = (4 if x["rank"] < ranks[3] else 8) * MiB       # a three-against-three tie
        keep = rng.random(len(g)) > 0.05
        recs += [x for x, k in zip(g, keep) if k or x["seq"] == 0]
    recs = [x for x in recs if not (x["comm"] == 1 and x["seq"] == 3)]                        # an op nobody reported
    an, o = hand_pair(recs, comms)
    keys = ("n_members", "n_present", "n_deviating_total", "majority_count", "op", "algo", "proto", "bytes")

    def check():
        for cid, ranks, _ in comms:
            for s in (0, 1, 2, 3, 4, 9):
                a, b = an.opset_check(0, cid, s), o.opset_check(0, cid, s)
                assert [a[k] for k in keys] == [b[k] for k in keys], (cid, s, a, b)
                assert np.array_equal(a["ranks"], b["ranks"]), (cid, s)
        short = an.opset_check(0, 3, 2, ranks_cap=3)
        assert len(short["ranks"]) == 3 and short["n_deviating_total"] == o.opset_check(0, 3, 2)["n_deviating_total"]

    check()
    assert an.opset_check(0, 0, 0)["n_deviating_total"] == 0 and an.opset_check(0, 3, 1)["n_deviating_total"] > 100
    algo = rng.integers(0, 2, len(recs)).astype(np.uint8); proto = (rng.random(len(recs)) < 0.1).astype(np.uint8)
    an.trace_attach_opset(0, algo, proto); assert o.attach_opset(0, algo, proto) == 0
    check()
    an.trace_attach_opset(0, torch.from_numpy(proto).cuda(), torch.from_numpy(algo).cuda())   # device columns, swapped
    assert o.attach_opset(0, proto, algo) == 0
    check()


def test_a_silent_rank_sends_every_group_of_its_communicators_to_the_general_path():
    """One rank reports nothing and another one's ops are all in flight: every group of their communicators is incomplete,
    so whole work units of the fused kernel are handed to the kernel for irregular groups, next to communicators that
    stay on the fast path. Windows start 30 s apart, so op times also cross many 2^32 ns boundaries."""
    spec = tg.cfg2(reps=40, n_windows=2, tp=8, pp=2, dp=16)
    spec.t0_ns = 30_000_000_000
    an, o = make_pair(tg.registry(spec))
    silent, stuck = 5, 77
    for w in range(2):
        win = tg.gen_window(spec, w, device="cuda")
        keep = win.cols["rank"] != silent
        cols = {k: v[keep].clone() for k, v in win.cols.items()}
        cols["t_exit"][cols["rank"] == stuck] = -1
        an.trace_upload(w, cols); assert o.upload(w, cols) == 0
        now = win.now_ns
    an.analyze_window(0, 2, now); assert o.analyze(0, 2, now) == 0
    for w in range(2):
        v, _ = compare_window(an, o, w)
        assert v["n_incomplete"] > 0 and v["n_complete"] > 0
    compare_cumulative(an, o, spec.n_ranks, 1)


@pytest.mark.parametrize("seed", [101, 102, 103])
def test_randomized_groups_with_random_damage(seed):
    """Seeded random communicators of 2 to 128 ranks over two windows with every kind of irregularity sprinkled in at random
    - missing records, ops in flight, exits before enters, negative times, spreads beyond 2^32 ns, barriers, differing
    sizes and ops - so that regular and irregular groups share warps and work units of the fused kernel."""
    rng = np.random.default_rng(seed)
    sizes = [int(x) for x in rng.choice([2, 3, 5, 8, 8, 8, 9, 16, 24, 32, 33, 64, 64, 100, 128], size=9)]
    recs, comms, r0 = [[], []], [], 0
    for cid, n in enumerate(sizes):
        ranks = [int(x) for x in (r0 + rng.permutation(n))]; r0 += n
        comms.append((cid * 3 + 1, ranks, 5))
        n_seq = int(rng.integers(20, 90))
        for w in range(2):
            durs = rng.integers(900_000, 1_300_000, size=(n_seq, n)).tolist()
            ents = rng.integers(0, 60_000, size=(n_seq, n)).tolist()
            g = group_trace(durs, ents, comm=cid * 3 + 1, ranks=ranks, seq0=5 + w * n_seq, t0=3_000_000_000 + w * 40_000_000_000,
                            spacing=int(rng.choice([7_000_000, 900_000_000])), bytes=4 * MiB)
            for r in g:
                u = rng.random()
                if u < 0.010: r["drop"] = True
                elif u < 0.015: r["t_exit"] = -1
                elif u < 0.020: r["t_exit"] = r["t_enter"] - 7
                elif u < 0.023: r["t_enter"] = -r["t_enter"]
                elif u < 0.028: r["t_exit"] += 6_000_000_000
                elif u < 0.033: r["t_enter"] -= 2_500_000_000
                elif u < 0.040: r["bytes"] = 8 * MiB
                elif u < 0.045: r["op"] = ALLGATHER
                r["send_chg"] = int(rng.integers(0, 9)); r["recv_chg"] = int(rng.integers(0, 9))
            for s in rng.choice(n_seq, size=2, replace=False):
                for r in g:
                    if r["seq"] == 5 + w * n_seq + int(s): r["bytes"] = 2          # a barrier
            recs[w] += [r for r in g if not r.pop("drop", False)]
    an, o = make_pair(comms)
    for w in range(2):
        order = rng.permutation(len(recs[w]))
        cols = make_cols([recs[w][i] for i in order])
        an.trace_upload(w, cols); assert o.upload(w, cols) == 0
    now = 3_000_000_000 + 500 * 10**9
    an.analyze_window(0, 2, now); assert o.analyze(0, 2, now) == 0
    for w in range(2):
        v, _ = compare_window(an, o, w)
        assert v["n_incomplete"] > 0 and v["n_complete"] > 0 and v["n_alerts_total"] > 0
    compare_cumulative(an, o, r0, 1)


# ---------------------------------------------------------------- tree communicators (Sec. 4.2.1: same-layer comparison)
@pytest.mark.gpu
def test_tree_communicators_compare_progress_within_a_layer():
    """Hung tree communicators of several sizes, layers as the depth of a binary tree or as random ids, counter totals
    that differ from layer to layer with random laggards, ties and missing frames: H3 names the same member as the
    oracle, through ccld_locate_hang and through the sweep; H1 / H2 and the per-op results do not depend on the layers."""
    rng = np.random.default_rng(77)
    C_ = 2
    an, o = ccld.Analyzer(), orc.Oracle()
    recs, entries, r0 = [], [], 0
    plan = [(7, "depth", "lag"), (7, "depth", "even"), (40, "rand", "lag"), (130, "depth", "tie"), (1500, "rand", "lag"),
            (3000, "depth", "lag"), (9, "depth", "h1"), (12, "rand", "h2"), (33, "one", "lag"), (20, "each", "lag")]
    for cid, (n, lay, kind) in enumerate(plan):
        ranks = (r0 + rng.permutation(n)).tolist(); r0 += n
        layers = {"depth": np.floor(np.log2(np.arange(n) + 1)).astype(np.uint32), "rand": rng.integers(0, 5, n).astype(np.uint32) * 1000 + 7,
                  "one": np.zeros(n, np.uint32), "each": np.arange(n, dtype=np.uint32)[::-1].copy()}[lay]
        an.comm_register(cid, ranks, 1, 0); assert o.comm_register(cid, ranks, 0) == 0
        an.comm_set_layers(cid, layers); assert o.comm_set_layers(cid, layers) == 0
        entered = set(range(n)) - ({1, n - 1} if kind == "h1" else set())
        done = {2, 3} if kind == "h2" else set()
        for r in hang_records(n, 1 + cid % 3, entered, done, ranks):
            r["comm"] = cid
            recs.append(r)
        tot = 50 + 10 * (layers % 13).astype(np.int64)                           # every layer has its own level
        if kind in ("lag", "tie", "h1", "h2"):
            k = max(1, n // 10)
            who = rng.choice(n, k, replace=False)
            tot[who] -= 9 if kind == "tie" else rng.integers(1, 40, k)           # "tie": the same gap in several layers
        for i in range(n):
            if n > 100 and i == n // 3: continue                                 # no frame: counts as zero
            entries.append((ranks[i], cid, 1 + cid % 3, [(int(tot[i]) // 2, int(tot[i]) - int(tot[i]) // 2)] * C_))
    cols = make_cols(recs)
    fr = frames_from(entries, C_)
    an.trace_upload(0, cols, fr, C_); assert o.upload(0, cols, fr, C_) == 0
    now = 10**9 + 400 * 10**9
    an.analyze_window(0, 1, now); assert o.analyze(0, 1, now) == 0
    compare_window(an, o, 0)
    sweep = an.locate_hangs(0, cap=32, roots_stride=16)
    assert len(sweep) == len(plan)
    seen = {}
    for d in sweep:
        b = o.locate_hang(0, d["comm"], d["seq"])
        a = an.locate_hang(0, d["comm"], d["seq"])
        for v in (d, a):
            assert v["cls"] == b["cls"] and v["n_roots_total"] == b["n_roots"], (v, b)
            for k in ("n_not_entered", "n_hung", "n_not_hung", "n_missing_frames", "stuck_step", "n_members", "min_total"):
                assert v[k] == b[k], (d["comm"], k, v[k], b[k])
            assert np.array_equal(v["roots"][:16], b["roots"][:16])
        seen[d["comm"]] = (b["cls"], b["n_roots"])
    assert seen[1] == (3, 0) and seen[9] == (3, 0)                              # layers that agree / of one member each: nobody
    assert seen[6][0] == 1 and seen[7][0] == 2 and all(seen[c] == (3, 1) for c in (0, 2, 3, 4, 5, 8))


@pytest.mark.gpu
def test_tree_communicator_call_order_and_errors():
    an = ccld.Analyzer()
    an.comm_register(0, [0, 1, 2], 0, 0); an.comm_register(1, [3, 4, 5], 1, 0); an.comm_register(2, [6, 7, 8], 1, 0)
    with pytest.raises(ccld.CcldError) as e:
        an.comm_register(3, [9, 10], 2, 0)
    assert e.value.code == -1
    with pytest.raises(ccld.CcldError) as e:
        an.comm_set_layers(0, [0, 1, 1])                                         # a ring has no layers
    assert e.value.code == -1
    with pytest.raises(ccld.CcldError) as e:
        an.comm_set_layers(9, [0])
    assert e.value.code == -4
    an.comm_set_layers(1, [0, 1, 1])
    recs = []
    for cid, ranks in ((1, [3, 4, 5]), (2, [6, 7, 8])):
        for r in hang_records(3, 0, {0, 1, 2}, set(), ranks):
            r["comm"] = cid; recs.append(r)
    an.trace_upload(0, make_cols(recs), frames_from([(4, 1, 0, [(5, 5)]), (5, 1, 0, [(2, 2)])], 1), 1)
    an.analyze_window(0, 1, 10**9 + 400 * 10**9)
    v = an.locate_hang(0, 1, 0)
    assert v["cls"] == 3 and list(v["roots"]) == [5] and v["min_total"] == 4 and v["stuck_step"] == 2
    with pytest.raises(ccld.CcldError) as e:
        an.locate_hang(0, 2, 0)                                                  # a tree whose layers were never set
    assert e.value.code == -9
    with pytest.raises(ccld.CcldError) as e:
        an.locate_hangs(0, cap=8, roots_stride=4)
    assert e.value.code == -9
    with pytest.raises(ccld.CcldError) as e:
        an.comm_set_layers(2, [0, 1, 1])                                         # too late
    assert e.value.code == -9


@pytest.mark.gpu
@pytest.mark.parametrize("with_rates", [True, False])
def test_tree_communicators_slow_root_compares_rates_within_a_layer(with_rates):
    """Slowed tree communicators of every kernel class over a batch of two windows: the communication root is the member
    that changes most often above its own layer's fewest changes (or the longest duration when no layer disagrees with
    itself, or without rate columns), identical to the oracle; a ring in the same batch keeps the ring rule."""
    rng = np.random.default_rng(5)
    params = dict(tbase_init_ns=2 * 10**6)
    an, o = ccld.Analyzer(params), orc.Oracle(params)
    plan = [(7, "depth", "lag"), (8, "rand", "even"), (40, "rand", "lag"), (130, "depth", "tie"), (1500, "rand", "lag"),
            (3000, "depth", "lag"), (33, "one", "lag"), (20, "each", "lag"), (16, None, "lag")]
    regs, r0 = [], 0
    for cid, (n, lay, kind) in enumerate(plan):
        ranks = (r0 + rng.permutation(n)).tolist(); r0 += n
        an.comm_register(cid, ranks, 0 if lay is None else 1, 0); assert o.comm_register(cid, ranks, 0) == 0
        layers = None
        if lay is not None:
            layers = {"depth": np.floor(np.log2(np.arange(n) + 1)).astype(np.uint32), "rand": rng.integers(0, 5, n).astype(np.uint32) * 1000 + 7,
                      "one": np.zeros(n, np.uint32), "each": np.arange(n, dtype=np.uint32)[::-1].copy()}[lay]
            an.comm_set_layers(cid, layers); assert o.comm_set_layers(cid, layers) == 0
        regs.append((ranks, layers, kind))
    wins = []
    for w in range(2):
        recs = []
        for cid, (ranks, layers, kind) in enumerate(regs):
            n = len(ranks)
            lv = (layers % 13).astype(np.int64) if layers is not None else np.zeros(n, np.int64)
            for s in range(3):
                chg = 3 + 2 * lv                                                # every layer has its own level
                if kind in ("lag", "tie"):
                    who = rng.choice(n, max(1, n // 10), replace=False)
                    chg = chg.copy(); chg[who] += 4 if kind == "tie" else rng.integers(1, 30, len(who))
                dur = 10**7 + rng.integers(0, 10**5, n) + (s == 1) * rng.integers(0, 10**6, n)   # op 1 has the widest range
                t0 = 10**9 * (1 + w) + s * 10**8
                for i in range(n):
                    recs.append(dict(rank=ranks[i], comm=cid, seq=3 * w + s, t_enter=t0, t_exit=t0 + int(dur[i]),
                                     send_chg=int(chg[i]) if i % 2 else 1, recv_chg=1 if i % 2 else int(chg[i])))
        wins.append(make_cols(recs, with_rates))
    for w in range(2):
        an.trace_upload(w, wins[w]); assert o.upload(w, wins[w]) == 0
    an.analyze_window(0, 2, 10**12); assert o.analyze(0, 2, 10**12) == 0
    for w in range(2):
        compare_window(an, o, w)
        rows = o.comm_rows(w)
        assert rows["slow_detected"].all() and (rows["sel_seq"] == 3 * w + 1).all()
        src = rows["rate_source"].tolist()
        assert src == ([0, 1, 0, 0, 0, 0, 0, 1, 0] if with_rates else [1] * 9)


# ---------------------------------------------------------------- batches enqueued without waiting for their plan
def test_repeated_shape_is_enqueued_without_waiting_and_stays_in_order():
    """Windows analysed one call at a time: from the second call on the shape is known, the call sizes its buffers from
    the earlier totals and only enqueues. Results, and the state that carries from window to window (Eq. 1 baseline going
    dynamic, the repetition counter), are those of the oracle walking the windows in order."""
    spec = tg.cfg2(reps=60, n_windows=6, tp=8, pp=2, dp=16)
    params = dict(m_max_rounds=150, tbase_init_ns=100_000)       # the baseline freezes in the second window, slow rounds repeat
    reg = tg.registry(spec)
    an, o = make_pair(reg, params)
    wins = [tg.gen_window(spec, w, device="cuda") for w in range(spec.n_windows)]
    for w, win in enumerate(wins):
        an.trace_upload(w, win.cols); assert o.upload(w, win.cols) == 0
    now = wins[-1].now_ns
    for w in range(spec.n_windows):
        an.analyze_window(w, 1, now)                             # nothing is read back in between
    assert o.analyze(0, spec.n_windows, now) == 0
    for w in range(spec.n_windows):
        compare_window(an, o, w)
    rows = o.comm_rows(spec.n_windows - 1)
    assert (rows["baseline_static"] == 0).any() and (rows["slow_count"] > 1).any()
    compare_cumulative(an, o, spec.n_ranks, spec.n_windows - 1)


@pytest.mark.parametrize("speculate", [True, False])
def test_a_batch_that_does_not_match_its_expected_layout_is_analysed_again_in_order(speculate):
    """Window 2 has the record count of its predecessors but one record with a far later op counter, so its layout (more
    groups, more slots) is not the one the call expected; windows 3 and 4 are enqueued behind it before anything is read
    back. All of them must come out as if every call had waited: same rows, same cumulative state, same order."""
    spec = tg.cfg2(reps=40, n_windows=5, tp=8, pp=2, dp=16)
    params = dict(m_max_rounds=100, tbase_init_ns=100_000)
    reg = tg.registry(spec)
    an, o = make_pair(reg, params)
    an.set_speculation(speculate)
    cols = []
    for w in range(spec.n_windows):
        c = {k: v.clone() for k, v in tg.gen_window(spec, w, device="cpu").cols.items()}
        if w == 2:
            c["seq"][7] += 500                                   # a rank far ahead: 500 groups nobody else reported
        cols.append(c)
    for w, c in enumerate(cols):
        an.trace_upload(w, c); assert o.upload(w, c) == 0
    now = tg.gen_window(spec, spec.n_windows - 1).now_ns
    an.timing_enable(True)
    for w in range(spec.n_windows):
        an.analyze_window(w, 1, now)
    assert o.analyze(0, spec.n_windows, now) == 0
    v2 = an.get_verdict(2, check=False)
    # the layout kernel runs twice per analysed batch: five calls, and - when calls do not wait - windows 2, 3 and 4 once more
    assert an.get_kernel_times()["k_plan"]["launches"] == (16 if speculate else 10)
    an.timing_enable(False)
    assert v2["n_incomplete"] == o.sizes(2)["n_incomplete"] > 400 and v2["n_groups"] == o.sizes(2)["n_groups"] > o.sizes(1)["n_groups"] + 400
    for w in range(spec.n_windows):
        compare_window(an, o, w)
    compare_cumulative(an, o, spec.n_ranks, spec.n_windows - 1)
    # the library keeps working in the same context: a reset and the same windows once more, now all as one batch
    an.reset()
    an.analyze_window(0, spec.n_windows, now)
    for w in range(spec.n_windows):
        compare_window(an, o, w)


def mismatching_windows(spec):
    """The windows of `spec` on the CPU; window 2 keeps its record count but carries one record with a far later op counter."""
    cols = []
    for w in range(spec.n_windows):
        c = {k: v.clone() for k, v in tg.gen_window(spec, w, device="cpu").cols.items()}
        if w == 2:
            c["seq"][7] += 500
        cols.append(c)
    return cols


def test_state_exported_while_batches_wait_is_the_state_after_all_of_them():
    """Calls that did not wait, one of them with a layout other than the expected one, and then - before any result is
    read - the cumulative state is exported and carried to a fresh context together with one more window. What arrives
    there must be the state after all five windows, in order: the export has to settle what is still waiting first."""
    spec = tg.cfg2(reps=40, n_windows=6, tp=8, pp=2, dp=16)
    params = dict(m_max_rounds=100, tbase_init_ns=100_000)
    reg = tg.registry(spec)
    an_a, o = make_pair(reg, params)
    an_b, _ = make_pair(reg, params)
    cols = mismatching_windows(spec)
    for w in range(5):
        an_a.trace_upload(w, cols[w]); assert o.upload(w, cols[w]) == 0
    an_b.trace_upload(5, cols[5]); assert o.upload(5, cols[5]) == 0
    now = tg.gen_window(spec, spec.n_windows - 1).now_ns
    for w in range(5):
        an_a.analyze_window(w, 1, now)
    blob = an_a.state_export()                                   # nothing was read back before this
    an_b.state_import(blob)
    an_b.analyze_window(5, 1, now)
    assert o.analyze(0, 6, now) == 0
    compare_window(an_b, o, 5)
    compare_cumulative(an_b, o, spec.n_ranks, 5)
    for w in range(5):
        compare_window(an_a, o, w)


def test_reset_and_release_while_batches_wait():
    """A reset right behind calls that did not wait discards them (also the one that would have had to be analysed again);
    a window released while its batch waits is settled first and the windows of the same batch stay readable."""
    spec = tg.cfg2(reps=40, n_windows=5, tp=8, pp=2, dp=16)
    params = dict(m_max_rounds=100, tbase_init_ns=100_000)
    reg = tg.registry(spec)
    an, o = make_pair(reg, params)
    cols = mismatching_windows(spec)
    for w, c in enumerate(cols):
        an.trace_upload(w, c); assert o.upload(w, c) == 0
    now = tg.gen_window(spec, spec.n_windows - 1).now_ns
    for w in range(spec.n_windows):
        an.analyze_window(w, 1, now)
    an.reset()                                                   # windows 2 to 4 were waiting to be analysed again
    for w in range(spec.n_windows):
        an.analyze_window(w, 1, now)
    an.window_release(3)                                         # its batch gave up behind window 2 and is still waiting
    assert o.analyze(0, spec.n_windows, now) == 0
    for w in (0, 1, 2, 4):
        compare_window(an, o, w)
    compare_cumulative(an, o, spec.n_ranks, 4)
    with pytest.raises(ccld.CcldError):
        an.get_verdict(3)
