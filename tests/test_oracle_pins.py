"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test is chosen so that a plausible slip in the oracle (a dropped term, a wrong sign or index,
an off-by-one median, a swapped class) fails it.
"""
import json
import os

import numpy as np
import pytest

import oracle as orc
from helpers import (ALLGATHER, ALLREDUCE, MiB, SENDRECV, frames_from, group_trace, make_cols)

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.json")))


def run(recs, comms, params=None, now=10**12, with_rates=True, frames=None, n_channels=0, windows=None):
    o = orc.Oracle(params)
    for cid, ranks, seq0 in comms:
        assert o.comm_register(cid, ranks, seq0) == 0
    if windows is None:
        windows = [recs]
    for w, r in enumerate(windows):
        assert o.upload(w, make_cols(r, with_rates), frames if w == len(windows) - 1 else None, n_channels) == 0
    assert o.analyze(0, len(windows), now) == 0
    return o


# ---------------------------------------------------------------- defaults the paper prints
def test_defaults_match_paper():
    p = orc.DEFAULT_PARAMS
    assert p["alpha_milli"] == round(GOLD["alpha"]["value"] * 1000)
    assert p["beta_milli"] == round(GOLD["beta"]["value"] * 1000)
    assert p["theta_slow_milli"] == GOLD["theta_slow"]["value"] * 1000
    assert p["m_max_rounds"] == GOLD["m_max_rounds"]["value"]
    assert p["m_max_ns"] == GOLD["m_max_seconds"]["value"] * 10**9
    assert p["hang_ns"] == GOLD["hang_threshold_seconds"]["value"] * 10**9
    assert p["barrier_bytes"] == GOLD["barrier_bytes"]["value"]
    f = GOLD["frame_bytes"]
    assert f["header"] + f["body"] == f["total"]
    # one block = Trace ID + channels x {SendCount, RecvCount} 8-byte slots
    assert f["body"] // f["blocks"] == f["trace_id"] + f["channels"] * 2 * 8


# ---------------------------------------------------------------- per-op quantities
def test_identical_ranks_flag_nothing():
    recs = group_trace([[2_000_000] * 8 for _ in range(20)])
    o = run(recs, [(0, list(range(8)), 0)])
    s = o.sizes(0)
    assert s["n_groups"] == 20 and s["n_complete"] == 20 and s["n_analysed"] == 20
    assert s["n_flag_skew"] == 0 and s["n_flag_dur"] == 0
    flags, _ = o.slots(0)
    assert (flags == 0).all()
    g = o.groups(0)
    assert (g["arrival_skew"] == 0).all() and (g["mad_dur"] == 0).all() and (g["med_dur"] == 2_000_000).all()
    assert o.suspects()["n_total"] == 0


def test_one_delayed_rank_is_the_only_one_flagged():
    rng = np.random.default_rng(1)
    durs, ents = [], []
    for s in range(50):
        durs.append([2_000_000 + int(x) for x in rng.integers(-1000, 1000, 8)])
        e = [3000 * ((i + s) % 8) for i in range(8)]           # evenly spread arrivals: nobody is an outlier
        e[5] += 2_000_000
        ents.append(e)
    o = run(group_trace(durs, ents), [(0, list(range(8)), 0)])
    flags, _ = o.slots(0)
    f = flags.reshape(50, 8)
    assert ((f[:, 5] & 1) == 1).all() and ((f[:, 5] & 4) == 4).all()     # late and above the median
    others = np.delete(f, 5, axis=1)
    assert ((others & 1) == 0).all()
    sus = o.suspects()
    assert list(sus["rank"][sus["kind"] == 1]) == [5]
    st = o.rank_stats(8)
    assert st["votes"][5, 0] == 50 and st["ops"][5] == 50


def test_hand_sets_median_mad():
    # {1,2,3,4,100}: lower median 3, deviations {2,1,0,1,97} -> MAD 1, only 100 is an outlier
    # {10,20,30,40}: lower median 20, deviations {10,0,10,20} -> sorted {0,10,10,20}, MAD 10, nobody flagged
    a = [[1, 2, 3, 4, 100]]
    b = [[10, 20, 30, 40]]
    o = run(group_trace(a, comm=0) + group_trace(b, comm=1), [(0, list(range(5)), 0), (1, list(range(4)), 0)])
    g = o.groups(0)
    assert list(g["med_dur"]) == [3, 20] and list(g["mad_dur"]) == [1, 10]
    assert list(g["t_max"]) == [100, 40] and list(g["t_min"]) == [1, 10]
    assert list(g["rank_tmax"]) == [4, 3] and list(g["rank_tmin"]) == [0, 0]
    flags, _ = o.slots(0)
    assert list(flags & 2) == [0, 0, 0, 0, 2, 0, 0, 0, 0]
    assert list(flags & 8) == [0, 0, 0, 8, 8, 0, 0, 8, 8]      # strictly above the median


def test_threshold_is_exact_integer_test():
    # n = 5 durations {0, 10, 20, 30, x}: median 20, deviations {20,10,0,10,x-20} -> MAD 10.
    # flag <=> (x-20)*1000 > k_milli*10. With k_milli = 5189: x-20 = 51 -> 51000 < 51890 no; 52 -> 52000 > 51890 yes.
    for x, want in ((71, 0), (72, 2)):
        o = run(group_trace([[0, 10, 20, 30, x]]), [(0, list(range(5)), 0)])
        flags, _ = o.slots(0)
        assert (flags[4] & 2) == want
    # equality is not an outlier: k_milli = 5000, deviation 50 -> 50000 > 50000 is false
    o = run(group_trace([[0, 10, 20, 30, 70]]), [(0, list(range(5)), 0)], params=dict(k_milli=5000))
    assert (o.slots(0)[0][4] & 2) == 0


def test_mad_zero_flags_any_deviation():
    o = run(group_trace([[7, 7, 7, 7, 7, 7, 7, 9]]), [(0, list(range(8)), 0)])
    flags, _ = o.slots(0)
    assert list(flags & 2) == [0] * 7 + [2]
    assert o.groups(0)["mad_dur"][0] == 0


def brute_order_stat(x, k):
    """k-th smallest by counting: the v in x with #{x < v} <= k < #{x <= v}."""
    for v in x:
        if sum(1 for y in x if y < v) <= k < sum(1 for y in x if y <= v):
            return v
    raise AssertionError


def test_median_mad_brute_force_by_counting():
    rng = np.random.default_rng(7)
    recs, comms = [], []
    sets = []
    for c, n in enumerate([4, 5, 6, 7, 8, 9, 13, 16, 31, 32, 33, 64, 100]):
        durs = [[int(v) for v in rng.integers(1, 50, n)] for _ in range(3)]      # many ties
        durs += [[int(v) for v in rng.integers(1, 2**40, n)] for _ in range(3)]
        ents = [[int(v) for v in rng.integers(0, 10**6, n)] for _ in range(6)]
        recs += group_trace(durs, ents, comm=c, ranks=list(range(1000 * c, 1000 * c + n)))
        comms.append((c, list(range(1000 * c, 1000 * c + n)), 0))
        sets += list(zip(durs, ents))
    o = run(recs, comms)
    g = o.groups(0)
    assert len(sets) == len(g["med_dur"])
    for i, (d, e) in enumerate(sets):
        n = len(d); k = (n - 1) // 2
        med = brute_order_stat(d, k)
        assert g["med_dur"][i] == med
        assert g["mad_dur"][i] == brute_order_stat([abs(v - med) for v in d], k)
        sk = [v - min(e) for v in e]
        meds = brute_order_stat(sk, k)
        assert g["med_skew"][i] == meds
        assert g["mad_skew"][i] == brute_order_stat([abs(v - meds) for v in sk], k)
        assert g["arrival_skew"][i] == max(sk) and min(sk) == 0
        assert g["t_min"][i] <= g["med_dur"][i] <= g["t_max"][i]


def test_mad_of_normal_sample_is_0_6745_sigma():
    rng = np.random.default_rng(3)
    n = 4001
    d = (10**9 + rng.normal(0, 10**6, n)).astype(np.int64)
    o = run(group_trace([[int(v) for v in d]]), [(0, list(range(n)), 0)])
    g = o.groups(0)
    assert abs(g["mad_dur"][0] / 10**6 - 0.6745) < 0.03
    assert abs(g["med_dur"][0] - 10**9) < 10**5


def test_bus_bandwidth_closed_forms():
    # allreduce, n = 8, 16 MiB: every rank enters at once and takes 2 ms -> 2(n-1)/n * bytes / t
    o = run(group_trace([[2_000_000] * 8]), [(0, list(range(8)), 0)])
    assert o.groups(0)["busbw"][0] == pytest.approx(16 * MiB * 14 / (2_000_000 * 8), rel=1e-15)
    assert o.groups(0)["busbw"][0] == pytest.approx(14.680064, rel=1e-12)
    # allgather (n-1)/n, sendrecv 1: span includes the arrival skew
    recs = group_trace([[1_000_000] * 4], [[0, 0, 0, 1_000_000]], comm=0, op=ALLGATHER, bytes=4 * MiB)
    recs += group_trace([[1_000_000] * 4], comm=1, ranks=[4, 5, 6, 7], op=SENDRECV, bytes=4 * MiB)
    o = run(recs, [(0, [0, 1, 2, 3], 0), (1, [4, 5, 6, 7], 0)])
    g = o.groups(0)
    assert g["span"][0] == 2_000_000
    assert g["busbw"][0] == pytest.approx(4 * MiB * 3 / (2_000_000 * 4), rel=1e-15)
    assert g["busbw"][1] == pytest.approx(4 * MiB / 1_000_000, rel=1e-15)
    st = o.rank_stats(8)
    assert st["bw_sum"][0] == pytest.approx(4 * MiB * 3 / (1_000_000 * 4), rel=1e-15) and st["bw_cnt"][0] == 1


def test_votes_total_equals_flag_total_and_invariants():
    import tracegen as tg
    spec = tg.cfg2(reps=40, n_windows=2, tp=4, pp=2, dp=4)
    o = orc.Oracle()
    for cid, ranks, seq0 in tg.registry(spec):
        o.comm_register(cid, ranks, seq0)
    tot_skew = tot_dur = 0
    for w in range(2):
        win = tg.gen_window(spec, w)
        o.upload(w, win.cols)
        o.analyze(w, 1, win.now_ns)
        s = o.sizes(w)
        flags, perm = o.slots(w)
        assert int((flags & 1).sum()) == s["n_flag_skew"] and int(((flags & 2) >> 1).sum()) == s["n_flag_dur"]
        assert s["n_groups"] == s["n_complete"] + s["n_incomplete"]
        tot_skew += s["n_flag_skew"]; tot_dur += s["n_flag_dur"]
        g = o.groups(w)
        assert (g["arrival_skew"] >= 0).all() and (g["t_min"] <= g["t_max"]).all()
        an = (g["gflags"] & 16) != 0                           # groups that went through the median test
        assert an.any() and not an.all()
        assert (g["t_min"][an] <= g["med_dur"][an]).all() and (g["med_dur"][an] <= g["t_max"][an]).all()
        assert (g["med_skew"][an] <= g["arrival_skew"][an]).all() and (g["med_dur"][~an] == 0).all()
        # e_min really is the smallest enter time of the group's records
        te = win.cols["t_enter"].numpy()
        for i in (0, 7, len(g["seq"]) - 1):
            n = int(g["n_present"][i]); s0 = int(g["slot0"][i])
            assert g["e_min"][i] == te[perm[s0:s0 + n]].min()
    st = o.rank_stats(spec.n_ranks)
    assert st["votes"][:, 0].sum() + st["votes"][:, 1].sum() == tot_skew
    assert st["votes"][:, 2].sum() + st["votes"][:, 3].sum() == tot_dur


# ---------------------------------------------------------------- grouping
def test_input_order_and_window_split_invariance():
    import tracegen as tg
    spec = tg.cfg2(reps=30, n_windows=1, tp=4, pp=2, dp=2)
    res = []
    for order in ("rank_major", "arrival", "shuffled"):
        o = orc.Oracle()
        for cid, ranks, seq0 in tg.registry(spec):
            o.comm_register(cid, ranks, seq0)
        win = tg.gen_window(spec, 0, order=order)
        o.upload(0, win.cols); o.analyze(0, 1, win.now_ns)
        g = o.groups(0)
        res.append((g, o.rank_stats(spec.n_ranks), o.slots(0)[0]))
    for g, st, fl in res[1:]:
        for k in g:
            assert np.array_equal(g[k], res[0][0][k]), k
        assert np.array_equal(st["votes"], res[0][1]["votes"]) and np.array_equal(fl, res[0][2])
        assert np.allclose(st["bw_sum"], res[0][1]["bw_sum"], rtol=1e-12)
    # splitting the same ops into two windows leaves the vote totals unchanged
    spec2 = tg.cfg2(reps=15, n_windows=2, tp=4, pp=2, dp=2)
    o = orc.Oracle()
    for cid, ranks, seq0 in tg.registry(spec2):
        o.comm_register(cid, ranks, seq0)
    for w in range(2):
        win = tg.gen_window(spec2, w)
        o.upload(w, win.cols)
    o.analyze(0, 2, win.now_ns)
    assert np.array_equal(o.rank_stats(spec.n_ranks)["votes"], res[0][1]["votes"])
    assert np.array_equal(o.rank_stats(spec.n_ranks)["ops"], res[0][1]["ops"])


def test_rejected_records_and_incomplete_groups():
    recs = group_trace([[5, 5, 5, 5], [5, 5, 5, 5], [5, 5, 5, 5]], seq0=10)
    recs = [r for r in recs if not (r["seq"] == 11 and r["rank"] == 2)]          # missing member
    recs.append(dict(rank=0, comm=99, seq=10, t_enter=1, t_exit=2))              # unknown communicator
    recs.append(dict(rank=77, comm=0, seq=10, t_enter=1, t_exit=2))              # not a member
    recs.append(dict(rank=1, comm=0, seq=3, t_enter=1, t_exit=2))                # before seq0
    o = run(recs, [(0, [0, 1, 2, 3], 10)])
    s = o.sizes(0)
    assert s["n_rejected"] == 3 and s["error_bits"] == 1 | 2 | 4
    assert s["n_groups"] == 3 and s["n_complete"] == 2 and s["n_incomplete"] == 1
    g = o.groups(0)
    assert list(g["n_present"]) == [4, 3, 4] and (g["gflags"][1] & 2) and g["t_max"][1] == 0
    flags, perm = o.slots(0)
    assert flags[6] == (64 | 128) and perm[6] == 0xFFFFFFFF and flags[5] == 128


def test_barrier_and_small_groups_are_not_analysed():
    recs = group_trace([[5, 5, 5, 900]], comm=0, bytes=3)                        # allreduce < 4 B: barrier
    recs += group_trace([[5, 5, 5, 900]], comm=1, ranks=[4, 5, 6, 7], bytes=4)   # exactly 4 B is not
    recs += group_trace([[5, 5, 900]], comm=2, ranks=[8, 9, 10])                 # below min_group
    recs += group_trace([[5, 5, 5, 900]], comm=3, ranks=[12, 13, 14, 15], op=ALLGATHER, bytes=3)
    o = run(recs, [(0, [0, 1, 2, 3], 0), (1, [4, 5, 6, 7], 0), (2, [8, 9, 10], 0), (3, [12, 13, 14, 15], 0)])
    g = o.groups(0)
    assert [int(f) & (4 | 16) for f in g["gflags"]] == [4, 16, 0, 16]
    flags, _ = o.slots(0)
    assert list(flags) == [128] * 4 + [0, 0, 0, 2 | 8] + [128] * 3 + [0, 0, 0, 2 | 8]
    assert o.sizes(0)["n_barrier"] == 1
    assert len(o.comm_rows(0)["comm"]) == 4 and o.comm_rows(0)["n_rounds"][0] == 0


def test_opset_mismatch():
    recs = group_trace([[5, 5, 5, 5]] * 2)
    recs[5]["bytes"] = 8 * MiB
    o = run(recs, [(0, [0, 1, 2, 3], 0)])
    assert [int(f) & 8 for f in o.groups(0)["gflags"]] == [0, 8]


# ---------------------------------------------------------------- Eq. 1-4 and slow location
MS = 1_000_000


def test_eq1_baseline_mean_of_first_m_rounds():
    # m_max_rounds = 3: baseline stays the configured value while r <= m, then floor(mean(Tmax of first 3))
    durs = [[10, 1], [21, 2], [30, 3], [40, 4]]
    p = dict(m_max_rounds=3, tbase_init_ns=1000, min_group=2)
    o = run(group_trace(durs[:3]), [(0, [0, 1], 0)], params=p)
    r = o.comm_rows(0)
    assert r["baseline_static"][0] == 1 and r["t_base"][0] == 1000 and r["m"][0] == 0
    o = run(group_trace(durs), [(0, [0, 1], 0)], params=p)
    r = o.comm_rows(0)
    assert r["baseline_static"][0] == 0 and r["m"][0] == 3 and r["t_base"][0] == (10 + 21 + 30) // 3 == 20
    # same rounds split over two windows: the state carries over
    o = run(None, [(0, [0, 1], 0)], params=p, windows=[group_trace(durs[:2]), group_trace(durs[2:], seq0=2)])
    assert o.comm_rows(0)["baseline_static"][0] == 1
    assert o.comm_rows(1)["t_base"][0] == 20 and o.comm_rows(1)["rounds_total"][0] == 4


def test_eq1_two_minute_rule():
    # rounds start 0 s, 50 s, 130 s after the first: only the first two fall inside 120 s
    recs = []
    for s, (t, d) in enumerate([(0, 10), (50 * 10**9, 13), (130 * 10**9, 99)]):
        for rk in (0, 1):
            recs.append(dict(rank=rk, comm=0, seq=s, t_enter=10**9 + t, t_exit=10**9 + t + d))
    o = run(recs, [(0, [0, 1], 0)])
    r = o.comm_rows(0)
    assert r["m"][0] == 2 and r["t_base"][0] == (10 + 13) // 2 and r["baseline_static"][0] == 0


def test_eq2_selects_round_with_largest_range_not_largest_time():
    # ranges: 100-90=10, 60-10=50, 60-10=50 (tie -> earliest), 200-199=1
    durs = [[100, 90, 95, 95], [60, 10, 30, 30], [10, 60, 30, 30], [200, 199, 199, 199]]
    o = run(group_trace(durs), [(0, [0, 1, 2, 3], 0)], params=dict(tbase_init_ns=10))
    r = o.comm_rows(0)
    assert r["sel_seq"][0] == 1 and r["t_max"][0] == 60 and r["t_min"][0] == 10
    assert r["R"][0] == pytest.approx((60 - 10) / 10) and r["slow_detected"][0] == 1
    assert r["n_rounds"][0] == 4


def test_eq3_threshold_strict():
    # T_base = 1000: R = 3.0 exactly is not slow, R just above is
    for tmax, want in ((4000, 0), (4001, 1)):
        o = run(group_trace([[tmax, 1000, 1000, 1000]]), [(0, [0, 1, 2, 3], 0)], params=dict(tbase_init_ns=1000))
        r = o.comm_rows(0)
        assert r["slow_detected"][0] == want and r["R"][0] == pytest.approx((tmax - 1000) / 1000)


def coupled(enter_off, own_dur, chg=None, seq=0):
    """Collective semantics: nobody leaves before the last rank arrived: t_exit = max enter + own duration."""
    last = max(enter_off)
    return [dict(rank=i, comm=0, seq=seq, t_enter=10**9 + seq * 10**9 + e, t_exit=10**9 + seq * 10**9 + last + d,
                 send_chg=(chg[i] if chg else 1), recv_chg=1) for i, (e, d) in enumerate(zip(enter_off, own_dur))]


def test_eq4_limits_of_p_and_root_ranks():
    lim = GOLD["p_limits"]
    p = dict(tbase_init_ns=2 * MS)
    comms = [(0, [0, 1, 2, 3], 0)]
    # computation-slow: rank 2 arrives 20 ms late -> the others wait; T_min -> T_base, P -> 1; root = min-duration rank
    o = run(coupled([0, 0, 20 * MS, 0], [2 * MS] * 4), comms, params=p)
    r = o.comm_rows(0)
    assert (r["t_max"][0], r["t_min"][0]) == (22 * MS, 2 * MS)
    assert r["P"][0] == pytest.approx(lim["comp_slow"]) and r["cls"][0] == 1 and r["root_comp"][0] == 2
    assert r["R"][0] == pytest.approx(10.0) and r["slow_detected"][0] == 1 and r["located"][0] == 0
    # communication-slow: everyone takes 5x as long, T_min -> T_max, P -> 0; root = most observed count changes
    o = run(coupled([0, 0, 0, 0], [10 * MS] * 4, chg=[2, 2, 2, 7]), comms, params=p)
    r = o.comm_rows(0)
    assert r["P"][0] == pytest.approx(lim["comm_slow"]) and r["cls"][0] == 2 and r["root_comm"][0] == 3 and r["rate_source"][0] == 0
    # equal contributions: T_max 18, T_min 10, T_base 2 -> P = 0.5 -> mixed, both roots reported
    o = run(coupled([0, 8 * MS, 0, 0], [10 * MS] * 4, chg=[9, 2, 2, 2]), comms, params=p)
    r = o.comm_rows(0)
    assert r["P"][0] == pytest.approx(lim["equal"]) and r["cls"][0] == 3
    assert r["root_comp"][0] == 1 and r["root_comm"][0] == 0


def test_alpha_beta_boundaries_are_strict():
    # T_base 1000, T_max 11000 -> den = 10000. P = 0.6 exactly -> mixed; 0.6001 -> comp; 0.4 -> mixed; 0.3999 -> comm
    for tmin, cls in ((5000, 3), (4999, 1), (7000, 3), (7001, 2)):
        o = run(group_trace([[11000, tmin, 8000, 8000]]), [(0, [0, 1, 2, 3], 0)], params=dict(tbase_init_ns=1000))
        assert o.comm_rows(0)["cls"][0] == cls, tmin


def test_send_rate_worked_example_and_duration_proxy():
    ex = GOLD["send_rate_example"]
    chg = [ex["normal_changes"]] * 3 + [ex["slow_changes"]]
    recs = coupled([0, 0, 0, 0], [10 * MS] * 4, chg=chg)
    o = run(recs, [(0, [0, 1, 2, 3], 0)], params=dict(tbase_init_ns=2 * MS))
    assert o.groups(0)["max_chg"][0] == 7 and o.comm_rows(0)["root_comm"][0] == 3     # rate 1/7 < 1/2
    # without rate columns the longest-duration rank stands in
    recs = group_trace([[10 * MS, 10 * MS, 12 * MS, 10 * MS]])
    o = run(recs, [(0, [0, 1, 2, 3], 0)], params=dict(tbase_init_ns=2 * MS), with_rates=False)
    r = o.comm_rows(0)
    assert r["rate_source"][0] == 1 and r["root_comm"][0] == 2


def test_repetition_counter_triggers_location_on_second_detection():
    p = dict(tbase_init_ns=2 * MS)
    w0 = coupled([0, 0, 20 * MS, 0], [2 * MS] * 4, seq=0)
    w1 = coupled([0, 0, 0, 0], [2 * MS] * 4, seq=1)            # a healthy window in between
    w2 = coupled([0, 20 * MS, 0, 0], [2 * MS] * 4, seq=2)
    o = run(None, [(0, [0, 1, 2, 3], 0)], params=p, windows=[w0, w1, w2])
    assert [int(o.comm_rows(w)["slow_detected"][0]) for w in range(3)] == [1, 0, 1]
    assert [int(o.comm_rows(w)["located"][0]) for w in range(3)] == [0, 0, 1]
    assert [int(o.comm_rows(w)["slow_count"][0]) for w in range(3)] == [1, 1, 2]
    assert o.comm_rows(2)["root_comp"][0] == 1


# ---------------------------------------------------------------- hang detection and location
def hang_records(n, seq, entered, done, t_enter=10**9):
    recs = []
    for s in range(seq):
        recs += [dict(rank=i, comm=0, seq=s, t_enter=1000 + s, t_exit=2000 + s) for i in range(n)]
    for i in range(n):
        if i in entered:
            recs.append(dict(rank=i, comm=0, seq=seq, t_enter=t_enter, t_exit=(t_enter + 5 if i in done else -1)))
    return recs


def test_hang_alert_threshold_and_barrier_filter():
    now = 10**9 + 300 * 10**9
    for extra, bytes_, want in ((1, 16 * MiB, 1), (0, 16 * MiB, 0), (1, 3, 0)):
        recs = hang_records(4, 2, {0, 1, 2, 3}, set())
        for r in recs:
            r["bytes"] = bytes_
        o = run(recs, [(0, [0, 1, 2, 3], 0)], now=now + extra)
        a = o.alerts(0)
        assert len(a["seq"]) == want
        if want:
            assert a["seq"][0] == 2 and a["age_ns"][0] == 300 * 10**9 + 1


def test_hang_tree_h1_not_entered():
    o = run(hang_records(6, 3, {0, 1, 2, 4}, set()), [(0, list(range(6)), 0)])
    h = o.locate_hang(0, 0, 3)
    assert h["cls"] == 1 and list(h["roots"]) == [3, 5] and h["n_not_entered"] == 2


def test_hang_tree_h2_non_hung_ranks():
    o = run(hang_records(6, 3, set(range(6)), {2}), [(0, list(range(6)), 0)])
    h = o.locate_hang(0, 0, 3)
    assert h["cls"] == 2 and list(h["roots"]) == [2] and h["n_hung"] == 5 and h["n_not_hung"] == 1


def test_hang_tree_h3_fewest_counts_and_ring_tie_break():
    n, C = 6, 2
    recs = hang_records(n, 3, set(range(n)), set())
    ranks = [10, 11, 12, 13, 14, 15]
    for r in recs:
        r["rank"] = ranks[r["rank"]]
    # unique minimum at ring position 4
    fr = frames_from([(ranks[i], 0, 3, [(9, 9), (9, 8)] if i != 4 else [(9, 7), (8, 6)]) for i in range(n)], C)
    o = run(recs, [(0, ranks, 0)], frames=fr, n_channels=C)
    h = o.locate_hang(0, 0, 3)
    assert h["cls"] == 3 and list(h["roots"]) == [14] and h["stuck_step"] == 6 and h["min_total"] == 30
    # a run of equal minima at positions 5,0,1 (wrapping): the most upstream one (5) is the root
    tot = {5: 4, 0: 4, 1: 4}
    fr = frames_from([(ranks[i], 0, 3, [(tot.get(i, 6), tot.get(i, 6))] * C) for i in range(n)], C)
    o = run(recs, [(0, ranks, 0)], frames=fr, n_channels=C)
    assert list(o.locate_hang(0, 0, 3)["roots"]) == [15]
    # all equal: lowest position; a missing frame counts as zero progress
    fr = frames_from([(ranks[i], 0, 3, [(5, 5)] * C) for i in range(n)], C)
    o = run(recs, [(0, ranks, 0)], frames=fr, n_channels=C)
    assert list(o.locate_hang(0, 0, 3)["roots"]) == [10]
    fr = frames_from([(ranks[i], 0, 3, [(5, 5)] * C) for i in range(n) if i != 2], C)
    o = run(recs, [(0, ranks, 0)], frames=fr, n_channels=C)
    h = o.locate_hang(0, 0, 3)
    assert list(h["roots"]) == [12] and h["n_missing_frames"] == 1 and h["min_total"] == 0


def test_windows_analysed_independently_add_up_to_the_sequential_run():
    """Votes, analysed-op counts and bandwidth sums are sums over windows: one fresh instance per window, four at a
    time, merged by addition, gives the statistics and the suspect list of one instance that saw the windows in order."""
    import tracegen as tg
    spec = tg.cfg2(reps=40, n_windows=5)
    reg = tg.registry(spec)
    wins = [tg.gen_window(spec, w) for w in range(spec.n_windows)]
    now = wins[-1].now_ns
    o = orc.Oracle()
    for cid, ranks, seq0 in reg:
        o.comm_register(cid, ranks, seq0)
    for w, win in enumerate(wins):
        o.upload(w, win.cols)
    o.analyze(0, len(wins), now)
    tot, sizes, n_rec = orc.analyze_windows_independently(reg, ((w, win.cols, now) for w, win in enumerate(wins)), spec.n_ranks, threads=4)
    assert n_rec == sum(w.n_rec for w in wins) and sorted(sizes) == list(range(5))
    ref = o.rank_stats(spec.n_ranks)
    for k in ("votes", "ops", "bw_cnt"):
        assert np.array_equal(ref[k], tot[k]), k
    assert np.allclose(ref["bw_sum"], tot["bw_sum"], rtol=1e-12, atol=0)
    for w in range(5):
        assert sizes[w]["n_flag_skew"] == o.sizes(w)["n_flag_skew"] and sizes[w]["n_groups"] == o.sizes(w)["n_groups"]
    merged = orc.Oracle()
    merged.add_rank_stats(tot)
    a, b = o.suspects(), merged.suspects()
    assert a["n_total"] == b["n_total"] > 0
    for k in ("kind", "rank", "votes", "ops"):
        assert np.array_equal(a[k], b[k]), k
    assert np.allclose(a["mean_busbw"], b["mean_busbw"], rtol=1e-12, atol=0)


# ---------------------------------------------------------------- branches of the grouping, hand cases
def test_invalid_times_make_the_group_incomplete():
    # op 0: rank 1 reports a negative enter time; op 1: rank 2 leaves before it entered; op 2 is healthy.
    recs = group_trace([[5, 5, 5, 5]] * 3)
    for r in recs:
        if r["seq"] == 0 and r["rank"] == 1:
            r["t_enter"], r["t_exit"] = -7, 3
        if r["seq"] == 1 and r["rank"] == 2:
            r["t_exit"] = r["t_enter"] - 1
    o = run(recs, [(0, [0, 1, 2, 3], 0)])
    s, g = o.sizes(0), o.groups(0)
    assert s["n_complete"] == 1 and s["n_incomplete"] == 2 and s["n_analysed"] == 1 and s["n_rejected"] == 0 and s["n_alerts"] == 0
    # bit 7 of the group word = invalid time, bit 1 = incomplete, bit 0 = complete; every member is present
    assert [int(f) & (1 | 2 | 64 | 128) for f in g["gflags"]] == [2 | 128, 2 | 128, 1]
    assert list(g["n_present"]) == [4, 4, 4]
    # an incomplete group carries no statistics, its records are present but not analysed, and it is no round of Eq. 1
    for k in ("e_min", "t_max", "t_min", "span", "med_dur", "arrival_skew"):
        assert list(g[k][:2]) == [0, 0], k
    flags, perm = o.slots(0)
    assert list(flags[:8]) == [128] * 8 and list(flags[8:]) == [0] * 4 and (perm != 0xFFFFFFFF).all()
    assert o.comm_rows(0)["n_rounds"][0] == 1 and o.comm_rows(0)["sel_seq"][0] == 2
    st = o.rank_stats(4)
    assert list(st["ops"]) == [1] * 4 and list(st["bw_cnt"]) == [1] * 4


def test_duplicate_record_keeps_the_first_and_counts_one_rejection():
    # rank 2 reports op 0 twice: 40 ns first, 900 ns second. The first one stands.
    recs = group_trace([[10, 20, 40, 30]])
    recs.append(dict(rank=2, comm=0, seq=0, t_enter=recs[2]["t_enter"], t_exit=recs[2]["t_enter"] + 900))
    o = run(recs, [(0, [0, 1, 2, 3], 0)])
    s, g = o.sizes(0), o.groups(0)
    assert s["n_rejected"] == 1 and s["error_bits"] == 8 and s["n_complete"] == 1 and s["n_slots"] == 4
    assert g["t_max"][0] == 40 and g["rank_tmax"][0] == 2 and g["n_present"][0] == 4
    assert list(o.slots(0)[1]) == [0, 1, 2, 3]
    # the other way round: the 900 ns record comes first in the upload and is the one kept
    recs = [recs[4]] + recs[:4]
    o = run(recs, [(0, [0, 1, 2, 3], 0)])
    assert o.groups(0)["t_max"][0] == 900 and o.sizes(0)["n_rejected"] == 1 and list(o.slots(0)[1]) == [1, 2, 0, 4]


def test_counter_range_comes_from_trace_ids_not_from_membership():
    # The Trace ID (Sec. 5.1) is communicator id + operation counter and carries no rank, so which operations a
    # communicator issued in a window is read off the Trace IDs alone. A record of rank 77, which is not a member,
    # names communicator 0 with counter 14 while the members report 10..11: the record is rejected, the operations
    # 12..14 exist and nobody reported them (incomplete, no member present). A counter below the communicator's first
    # (3 < 10) names no operation and widens nothing.
    recs = group_trace([[5, 5, 5, 5], [5, 5, 5, 5]], seq0=10)
    recs.append(dict(rank=77, comm=0, seq=14, t_enter=1, t_exit=2))
    recs.append(dict(rank=77, comm=0, seq=3, t_enter=1, t_exit=2))
    o = run(recs, [(0, [0, 1, 2, 3], 10)])
    s, g = o.sizes(0), o.groups(0)
    assert s["n_rejected"] == 2 and s["error_bits"] == 2
    assert list(g["seq"]) == [10, 11, 12, 13, 14] and s["n_slots"] == 20
    assert list(g["n_present"]) == [4, 4, 0, 0, 0] and s["n_complete"] == 2 and s["n_incomplete"] == 3
    assert [int(f) & 3 for f in g["gflags"]] == [1, 1, 2, 2, 2]
    flags, perm = o.slots(0)
    assert list(flags[8:]) == [64 | 128] * 12 and (perm[8:] == 0xFFFFFFFF).all()
    assert o.comm_rows(0)["n_rounds"][0] == 2
    # the same record from a member would have been accepted into op 14
    recs[-2]["rank"] = 1
    o = run(recs, [(0, [0, 1, 2, 3], 10)])
    assert list(o.groups(0)["n_present"]) == [4, 4, 0, 0, 1] and o.sizes(0)["n_rejected"] == 1


def test_barrier_groups_add_nothing_to_the_bandwidth_sums():
    # op 0: a 3-byte AllReduce (barrier), op 1: 16 MiB in 2 ms over 4 ranks: 16 MiB * 2*3/4 / 2e6 ns = 12.582912 GB/s
    recs = group_trace([[1000] * 4], bytes=3) + group_trace([[2 * MS] * 4], seq0=1, t0=2 * 10**9)
    o = run(recs, [(0, [0, 1, 2, 3], 0)])
    st = o.rank_stats(4)
    assert list(st["bw_cnt"]) == [1] * 4 and list(st["ops"]) == [1] * 4
    assert st["bw_sum"] == pytest.approx([16 * MiB * 6 / 4 / (2 * MS)] * 4, rel=1e-15)
    g = o.groups(0)
    assert g["busbw"][1] == pytest.approx(12.582912, rel=1e-15)
    assert g["busbw"][0] == pytest.approx(3 * 6 / 4 / 1000, rel=1e-15)      # the group value is still reported
    assert o.comm_rows(0)["n_rounds"][0] == 1                               # and a barrier is no round of Eq. 1 / Eq. 2


def test_eq1_two_minute_rule_at_the_boundary():
    # "all rounds within the first two minutes" (Sec. 4.2.1): a round that starts exactly 120 s after the first is
    # outside, one nanosecond earlier it is inside (and m stays open: 2 rounds < 100).
    for gap, m, base, static in ((120 * 10**9, 1, 10, 0), (120 * 10**9 - 1, 0, 2 * MS, 1)):
        recs = []
        for s, (t, d) in enumerate([(0, 10), (gap, 50)]):
            for rk in (0, 1):
                recs.append(dict(rank=rk, comm=0, seq=s, t_enter=10**9 + t, t_exit=10**9 + t + d))
        o = run(recs, [(0, [0, 1], 0)])
        r = o.comm_rows(0)
        assert (r["m"][0], r["t_base"][0], r["baseline_static"][0], r["rounds_total"][0]) == (m, base, static, 2), gap


def test_suspect_threshold_order_and_mean_bandwidth():
    # 8 ranks, 10 identical AllReduces of 16 MiB in 2 ms; late arrivals: rank 6 twice, ranks 3 and 1 once each;
    # rank 0 takes 4 ms once. Skews and durations are otherwise equal, so MAD = 0 and every deviation is flagged.
    durs = [[2 * MS] * 8 for _ in range(10)]
    ents = [[0] * 8 for _ in range(10)]
    ents[0][6] = ents[5][6] = 500_000
    ents[2][3] = 500_000
    ents[7][1] = 500_000
    durs[4][0] = 4 * MS
    o = run(group_trace(durs, ents), [(0, list(range(8)), 0)])
    st = o.rank_stats(8)
    assert list(st["votes"][:, 0]) == [0, 1, 0, 1, 0, 0, 2, 0] and list(st["votes"][:, 2]) == [1] + [0] * 7
    assert list(st["ops"]) == [10] * 8
    # votes * 1000 >= vote_rep_milli * ops with vote_rep_milli = 100: one vote in ten ops is exactly on the boundary
    sus = o.suspects()
    assert sus["n_total"] == 4
    assert list(sus["kind"]) == [1, 1, 1, 2]                 # stragglers first,
    assert list(sus["rank"]) == [6, 1, 3, 0]                 # more votes first, equal votes by rank
    assert list(sus["votes"]) == [2, 1, 1, 1] and list(sus["ops"]) == [10] * 4
    full = 16 * MiB * 14 / 8 / (2 * MS)                      # 14.680064 GB/s
    assert full == pytest.approx(14.680064, rel=1e-15)
    assert list(sus["mean_busbw"][:3]) == pytest.approx([full] * 3, rel=1e-12)
    assert sus["mean_busbw"][3] == pytest.approx((9 * full + full / 2) / 10, rel=1e-12)
    # one milli above the boundary the single-vote ranks drop out
    o = run(group_trace(durs, ents), [(0, list(range(8)), 0)], params=dict(vote_rep_milli=101))
    sus = o.suspects()
    assert list(sus["kind"]) == [1] and list(sus["rank"]) == [6]


def test_hang_tree_h1_counts_a_later_operation_counter_as_entered():
    # Leaf H1 names the members whose operation counter did not advance to the hung op (Sec. 4.2.2). Op 3 hangs:
    # ranks 0 and 1 are inside it, rank 2 has no record of op 3 but reports op 4 (its counter is past 3), rank 3 reports
    # nothing from op 3 on. Only rank 3 is named.
    recs = hang_records(4, 3, {0, 1}, set())
    recs.append(dict(rank=2, comm=0, seq=4, t_enter=10**9 + 10, t_exit=-1))
    o = run(recs, [(0, [0, 1, 2, 3], 0)])
    h = o.locate_hang(0, 0, 3)
    assert h["cls"] == 1 and list(h["roots"]) == [3] and h["n_not_entered"] == 1
    assert h["n_hung"] == 4 and h["n_not_hung"] == 0
    # asked about op 4 instead, ranks 0, 1 and 3 have not reached it
    h = o.locate_hang(0, 0, 4)
    assert h["cls"] == 1 and list(h["roots"]) == [0, 1, 3]


# ---------------------------------------------------------------- the benchmark configurations
def test_cfg1_rank5_is_the_sole_suspect():
    import tracegen as tg
    spec = tg.cfg1()
    o = orc.Oracle()
    for cid, ranks, seq0 in tg.registry(spec):
        o.comm_register(cid, ranks, seq0)
    win = tg.gen_window(spec, 0)
    o.upload(0, win.cols); o.analyze(0, 1, win.now_ns)
    s = o.sizes(0)
    assert s["n_records"] == 8000 and s["n_groups"] == 1000 and s["n_complete"] == 1000 and s["n_alerts"] == 0
    sus = o.suspects()
    assert sorted(set(sus["rank"])) == [5] and list(sus["kind"]) == [1]
    st = o.rank_stats(8)
    assert 250 <= st["votes"][5, 0] <= 350


def test_cfg3_hang_root_1793_step_23():
    import tracegen as tg
    spec = tg.cfg3()
    o = orc.Oracle()
    for cid, ranks, seq0 in tg.registry(spec):
        o.comm_register(cid, ranks, seq0)
    win = tg.gen_window(spec, 0)
    o.upload(0, win.cols, win.frames, win.n_channels); o.analyze(0, 1, win.now_ns)
    a = o.alerts(0)
    assert list(a["comm"]) == [7] and list(a["seq"]) == [100]
    h = o.locate_hang(0, 7, 100)
    assert h["cls"] == 3 and list(h["roots"]) == [1793] and h["stuck_step"] == 23
    assert h["min_total"] == 16 * 2 * 23 and h["n_hung"] == 256
    # a ring that completed: every rank is "not hung", which the tree reads as H2 with all ranks
    assert o.locate_hang(0, 3, 100)["cls"] == 2


def test_scaled_cfg2_and_cfg5_recover_injected_ranks():
    import tracegen as tg
    for spec in (tg.cfg2(reps=60, n_windows=2), tg.cfg5(reps=2, n_windows=2, nodes=64, mid=32, hang_window=1)):
        o = orc.Oracle()
        for cid, ranks, seq0 in tg.registry(spec):
            o.comm_register(cid, ranks, seq0)
        alerts = []
        for w in range(spec.n_windows):
            win = tg.gen_window(spec, w)
            o.upload(w, win.cols, win.frames, win.n_channels); o.analyze(w, 1, win.now_ns)
            a = o.alerts(w)
            alerts += [(w, int(c), int(s)) for c, s in zip(a["comm"], a["seq"])]
        sus = o.suspects()
        strag = sorted(set(int(r) for r in sus["rank"][sus["kind"] == 1]))
        slow = sorted(set(int(r) for r in sus["rank"][sus["kind"] == 2]))
        assert strag == spec.truth["stragglers"], (spec.name, strag)
        assert slow == spec.truth["slow_links"], (spec.name, slow)
        if spec.hang is not None:
            assert len(alerts) == 1
            w, c, s = alerts[0]
            h = o.locate_hang(w, c, s)
            assert h["cls"] == 3 and list(h["roots"]) == spec.truth["hang_root"] and h["stuck_step"] == 41


# ---------------------------------------------------------------- counter changes from raw probe samples (Sec. 4.1.2)
MS = 1_000_000


def _ticks(series):
    """series: per rank a list of (t_ns, send_count, recv_count) -> CSR arrays."""
    off = np.cumsum([0] + [len(s) for s in series]).astype(np.uint64)
    flat = [x for s in series for x in s]
    return (off, np.array([x[0] for x in flat], np.int64), np.array([x[1] for x in flat], np.uint32),
            np.array([x[2] for x in flat], np.uint32))


def test_derived_rates_reproduce_the_papers_worked_example():
    """Sec. 4.1.2, Fig. 5: probed every 1 ms, 8 sends show as 2 value changes on a normal rank and as 7 on a slow one."""
    ex = GOLD["send_rate_example"]
    normal = [(k * MS, min(8, 4 * k), 0) for k in range(11)]                      # 0, 4, 8, 8, ...
    slow_vals = [0, 1, 2, 3, 4, 6, 7, 8, 8, 8, 8]                                 # seven changes to reach 8
    slow = [(k * MS, slow_vals[k], 0) for k in range(11)]
    off, tn, sc, rc = _ticks([normal, slow])
    s, r = orc.derive_rates([0, 1], [0, 0], [10 * MS, 10 * MS], off, tn, sc, rc)
    assert list(s) == [ex["normal_changes"], ex["slow_changes"]] and list(r) == [0, 0]
    # the rate is the reciprocal of the count: 1/2 against 1/7
    assert [1, int(s[0])] == ex["normal_rate"] and [1, int(s[1])] == ex["slow_rate"]


def test_derived_rates_closed_form_boundaries_and_additivity():
    # a counter that advances at every tick: changes = ticks in (t_enter, t_exit]; recv advances every second tick
    T = 200
    ser = [(1000 + k * MS, k, k // 2) for k in range(T)]
    off, tn, sc, rc = _ticks([ser])
    rng = np.random.default_rng(11)
    a = rng.integers(0, T * MS, 64); b = a + rng.integers(0, 30 * MS, 64)
    s, r = orc.derive_rates(np.zeros(64, np.uint32), a, b, off, tn, sc, rc)
    tick = lambda t: np.clip((t - 1000) // MS + 1, 0, T)                           # ticks at or before t
    assert np.array_equal(s, np.maximum(tick(b), 1) - np.maximum(tick(a), 1))      # the rank's first tick never counts
    # a tick exactly at t_enter is outside, exactly at t_exit inside
    s2, _ = orc.derive_rates([0, 0], [1000 + 5 * MS, 1000 + 5 * MS - 1], [1000 + 7 * MS, 1000 + 7 * MS - 1], off, tn, sc, rc)
    assert list(s2) == [2, 2]
    # adjacent ops add up to the enclosing one
    cuts = np.sort(rng.integers(0, T * MS, 9))
    s3, r3 = orc.derive_rates(np.zeros(8, np.uint32), cuts[:-1], cuts[1:], off, tn, sc, rc)
    s4, r4 = orc.derive_rates([0], [cuts[0]], [cuts[-1]], off, tn, sc, rc)
    assert s3.sum() == s4[0] and r3.sum() == r4[0]
    # constant counters, an op in flight (counts to the end of the samples), a rank without samples, an unknown rank
    off2, tn2, sc2, rc2 = _ticks([[(k * MS, 5, 9) for k in range(50)], ser, []])
    s5, r5 = orc.derive_rates([0, 1, 2, 7], [0, 1000 + 150 * MS, 0, 0], [40 * MS, -1, 40 * MS, 40 * MS], off2, tn2, sc2, rc2)
    assert list(s5) == [0, T - 1 - 150, 0, 0] and list(r5) == [0, (T - 1) // 2 - 150 // 2, 0, 0]


def test_derived_rates_against_a_numpy_restatement():
    rng = np.random.default_rng(12)
    series = []
    for _ in range(9):
        n = int(rng.integers(0, 300))
        t = np.sort(rng.choice(400 * MS, size=n, replace=False))
        series.append(list(zip(t.tolist(), np.cumsum(rng.integers(0, 3, n)).tolist(), np.cumsum(rng.integers(0, 2, n)).tolist())))
    off, tn, sc, rc = _ticks(series)
    n_rec = 500
    rank = rng.integers(0, 9, n_rec).astype(np.uint32)
    te = rng.integers(0, 400 * MS, n_rec); tx = te + rng.integers(0, 50 * MS, n_rec)
    tx[rng.random(n_rec) < 0.05] = -1
    s, r = orc.derive_rates(rank, te, tx, off, tn, sc, rc)
    for i in range(n_rec):
        lo, hi = int(off[rank[i]]), int(off[rank[i] + 1])
        t = tn[lo:hi]
        inside = (t[1:] > te[i]) & ((t[1:] <= tx[i]) | (tx[i] == -1))
        assert s[i] == int((np.diff(sc[lo:hi].astype(np.int64))[inside] != 0).sum())
        assert r[i] == int((np.diff(rc[lo:hi].astype(np.int64))[inside] != 0).sum())


# ---------------------------------------------------------------- Operation Type Set consistency (Sec. 4.1.2, Sec. 4.2.2)
def _opset_oracle(recs, comms, algo=None, proto=None):
    o = orc.Oracle()
    for cid, ranks, seq0 in comms:
        assert o.comm_register(cid, ranks, seq0) == 0
    assert o.upload(0, make_cols(recs)) == 0
    if algo is not None:
        assert o.attach_opset(0, algo, proto) == 0
    return o


def test_opset_majority_hand_cases():
    ranks = [20, 21, 22, 23, 24, 25]
    recs = group_trace([[5] * 6] * 3, ranks=ranks)                                 # three ops, everyone agrees
    o = _opset_oracle(recs, [(0, ranks, 0)])
    r = o.opset_check(0, 0, 1)
    assert (r["n_members"], r["n_present"], r["n_deviating_total"], r["majority_count"]) == (6, 6, 0, 6) and r["bytes"] == 16 * MiB
    # one rank issues another size, one another operation, one has not reported: two deviants, ring order
    recs2 = [dict(x) for x in recs if not (x["seq"] == 1 and x["rank"] == 25)]
    for x in recs2:
        if x["seq"] == 1 and x["rank"] == 23: x["bytes"] = 8 * MiB
        if x["seq"] == 1 and x["rank"] == 21: x["op"] = ALLGATHER
    r = _opset_oracle(recs2, [(0, ranks, 0)]).opset_check(0, 0, 1)
    assert (r["n_present"], r["n_deviating_total"], r["majority_count"], r["op"]) == (5, 2, 3, ALLREDUCE) and list(r["ranks"]) == [21, 23]
    # algorithm / protocol columns: same op and size, two ranks on another protocol
    algo = np.zeros(len(recs), np.uint8); proto = np.zeros(len(recs), np.uint8)
    for i, x in enumerate(recs):
        if x["seq"] == 2 and x["rank"] in (20, 24): proto[i] = 2
    r = _opset_oracle(recs, [(0, ranks, 0)], algo, proto).opset_check(0, 0, 2)
    assert r["n_deviating_total"] == 2 and list(r["ranks"]) == [20, 24] and r["proto"] == 0 and r["majority_count"] == 4
    # a tie goes to the tuple whose first holder stands earliest in the ring: positions 0-2 against 3-5
    for i, x in enumerate(recs):
        proto[i] = 1 if (x["seq"] == 0 and x["rank"] >= 23) else proto[i]
    r = _opset_oracle(recs, [(0, ranks, 0)], algo, proto).opset_check(0, 0, 0)
    assert r["majority_count"] == 3 and r["proto"] == 0 and list(r["ranks"]) == [23, 24, 25]
    # an op nobody reported
    r = o.opset_check(0, 0, 9)
    assert (r["n_present"], r["n_deviating_total"], r["majority_count"]) == (0, 0, 0)


def test_opset_majority_against_a_counter_restatement():
    from collections import Counter
    rng = np.random.default_rng(31)
    n = 40
    ranks = list(rng.permutation(200)[:n].astype(int))
    recs = group_trace([[5] * n] * 6, ranks=ranks)
    for x in recs:
        x["op"] = int(rng.integers(0, 2)); x["bytes"] = int(rng.choice([4, 8])) * MiB
    keep = rng.random(len(recs)) > 0.1
    recs = [x for x, k in zip(recs, keep) if k]
    algo = rng.integers(0, 2, len(recs)).astype(np.uint8); proto = rng.integers(0, 2, len(recs)).astype(np.uint8)
    o = _opset_oracle(recs, [(0, ranks, 0)], algo, proto)
    for s in range(6):
        tup = {}
        for i, x in enumerate(recs):
            if x["seq"] == s: tup[x["rank"]] = (x["op"], x["bytes"], int(algo[i]), int(proto[i]))
        cnt = Counter(tup.values())
        top = max(cnt.values())
        maj = next(tup[r] for r in ranks if r in tup and cnt[tup[r]] == top)
        r = o.opset_check(0, 0, s)
        assert (r["op"], r["bytes"], r["algo"], r["proto"]) == maj and r["majority_count"] == top and r["n_present"] == len(tup)
        assert list(r["ranks"]) == [q for q in ranks if q in tup and tup[q] != maj]


# ---------------------------------------------------------------- tree communicators: same-layer comparison (Sec. 4.2.1)
def _tree_hang(tots, layers, ring=False, drop_frame=None):
    n = len(tots)
    ranks = list(range(50, 50 + n))
    recs = [dict(rank=r, comm=0, seq=0, t_enter=10**9, t_exit=-1) for r in ranks]
    entries = [(ranks[i], 0, 0, [(tots[i] // 2, tots[i] - tots[i] // 2)]) for i in range(n) if i != drop_frame]
    o = orc.Oracle()
    assert o.comm_register(0, ranks, 0) == 0
    if not ring:
        assert o.comm_set_layers(0, layers) == 0
    assert o.upload(0, make_cols(recs), frames_from(entries, 1), 1) == 0
    assert o.analyze(0, 1, 10**9 + 400 * 10**9) == 0
    return o.locate_hang(0, 0, 0), ranks


def test_tree_hang_root_is_compared_with_its_own_layer_only():
    layers = [0, 1, 1, 2, 2, 2, 2]
    # the tree's root forwards little (3) and every leaf agrees (10): a ring would blame position 0, the tree names the
    # layer-1 member that is 8 behind its peer
    tots = [3, 20, 12, 10, 10, 10, 10]
    h, ranks = _tree_hang(tots, layers, ring=True)
    assert h["cls"] == 3 and list(h["roots"]) == [ranks[0]]
    h, ranks = _tree_hang(tots, layers)
    assert h["cls"] == 3 and list(h["roots"]) == [ranks[2]] and h["min_total"] == 12 and h["stuck_step"] == 6
    # the largest gap inside a layer wins; equal gaps: the lowest position
    h, ranks = _tree_hang([3, 20, 12, 10, 1, 10, 10], layers)
    assert list(h["roots"]) == [ranks[4]] and h["min_total"] == 1
    h, ranks = _tree_hang([3, 20, 12, 10, 2, 10, 10], layers)
    assert list(h["roots"]) == [ranks[2]]
    h, ranks = _tree_hang([3, 12, 20, 10, 10, 2, 10], layers)
    assert list(h["roots"]) == [ranks[1]]
    # every layer agrees with itself: the counters name nobody
    h, ranks = _tree_hang([3, 20, 20, 10, 10, 10, 10], layers)
    assert h["cls"] == 3 and h["n_roots"] == 0 and len(h["roots"]) == 0 and h["min_total"] == 0
    # a member without a frame counts as zero and so lags its layer
    h, ranks = _tree_hang([3, 20, 20, 10, 10, 10, 10], layers, drop_frame=5)
    assert list(h["roots"]) == [ranks[5]] and h["n_missing_frames"] == 1 and h["stuck_step"] == 0


def _tree_slow(chg, layers, durs=None, with_rates=True):
    n = len(chg)
    ranks = list(range(70, 70 + n))
    durs = durs or [10 * MS] * n
    recs = [dict(rank=ranks[i], comm=0, seq=0, t_enter=10**9, t_exit=10**9 + durs[i], send_chg=chg[i], recv_chg=1) for i in range(n)]
    o = orc.Oracle(dict(tbase_init_ns=2 * MS))
    assert o.comm_register(0, ranks, 0) == 0
    if layers is not None:
        assert o.comm_set_layers(0, layers) == 0
    assert o.upload(0, make_cols(recs, with_rates)) == 0
    assert o.analyze(0, 1, 10**12) == 0
    r = o.comm_rows(0)
    assert r["slow_detected"][0] == 1
    return int(r["root_comm"][0]) - 70, int(r["rate_source"][0])


def test_tree_slow_root_compares_update_frequencies_within_a_layer():
    layers = [0, 1, 1, 2, 2, 2, 2]
    # the tree's root relays everything and changes most often (12): a ring would name it; inside the layers only
    # position 5 (6 changes against its layer's 3) stands out
    chg = [12, 6, 6, 3, 3, 6, 3]
    assert _tree_slow(chg, None) == (0, 0)
    assert _tree_slow(chg, layers) == (5, 0)
    # the larger excess wins; equal excesses: the lowest position
    assert _tree_slow([12, 6, 10, 3, 3, 6, 3], layers) == (2, 0)
    assert _tree_slow([12, 6, 9, 3, 3, 6, 3], layers) == (2, 0)
    assert _tree_slow([12, 9, 6, 3, 3, 3, 6], layers) == (1, 0)
    # every layer uniform: the rates name nobody and the longest duration stands in, as it does without rate columns
    durs = [10 * MS] * 7; durs[4] = 12 * MS
    assert _tree_slow([12, 6, 6, 3, 3, 3, 3], layers, durs) == (4, 1)
    assert _tree_slow(chg, layers, durs, with_rates=False) == (4, 1)
