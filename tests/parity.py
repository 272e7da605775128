"""Element-by-element comparison of the CUDA library with the CPU oracle on the same inputs."""
import numpy as np

import oracle as orc
import paper_2605_04478_b200 as ccld

REL = 1e-9   # tolerance for the fp64 quantities (bus bandwidths, R, P); everything else is bit-exact

INT_COLS = ("comm", "seq", "slot0") + ccld.OPTABLE_I64 + ccld.OPTABLE_U32


def make_pair(registry, params=None):
    an = ccld.Analyzer(params)
    o = orc.Oracle(params)
    for cid, ranks, seq0 in registry:
        an.comm_register(cid, ranks, 0, seq0)
        assert o.comm_register(cid, ranks, seq0) == 0
    return an, o


def close(a, b, what):
    a = np.asarray(a, dtype=np.float64); b = np.asarray(b, dtype=np.float64)
    assert a.shape == b.shape, what
    bad = np.abs(a - b) > REL * np.maximum(np.abs(a), np.abs(b))
    assert not bad.any(), (what, int(bad.sum()), a[bad][:4], b[bad][:4])


def same(a, b, what):
    a = np.asarray(a); b = np.asarray(b)
    assert a.shape == b.shape, (what, a.shape, b.shape)
    if not np.array_equal(a, b):
        i = np.nonzero(a != b)[0]
        raise AssertionError((what, len(i), i[:8], a[i[:8]], b[i[:8]]))


def compare_window(an, o, w, stateless_only=False, expect_rc=0):
    """Checks counts, the per-op table, flags, the slot permutation, communicator rows and alerts of window w."""
    v = an.get_verdict(w, check=False)
    s = o.sizes(w)
    assert v["rc"] == expect_rc, (v["rc"], expect_rc)
    for k in ("n_records", "n_groups", "n_slots", "n_rejected", "n_complete", "n_incomplete", "n_barrier", "n_analysed",
              "n_flag_skew", "n_flag_dur", "n_opset_mismatch", "error_bits"):
        assert v[k] == s[k], (k, v[k], s[k])
    assert v["n_comm_rows_total"] == s["n_comm_rows"] and v["n_alerts_total"] == s["n_alerts"]
    t = an.get_optable(w)
    g = o.groups(w)
    for k in INT_COLS:
        same(t[k], g[k], k)
    close(t["busbw"], g["busbw"], "busbw")
    flags, perm = o.slots(w)
    same(t["flags"], flags, "flags")
    # the oracle lists record indices group-major; the library stores them member-major inside each communicator
    r = an.get_ranges(w)
    want = perm.copy()
    for s0, n, ns in zip(r["slot0"].astype(np.int64), r["n"].astype(np.int64), r["n_seq"].astype(np.int64)):
        want[s0:s0 + n * ns] = perm[s0:s0 + n * ns].reshape(ns, n).T.reshape(-1)
    same(t["perm"], want, "perm")
    a, b = v["alerts"], o.alerts(w)
    ka = np.lexsort((a["seq"], a["comm"])); kb = np.lexsort((b["seq"], b["comm"]))
    for k in ("comm", "seq", "age_ns"):
        same(a[k][ka], b[k][kb], "alert " + k)
    if not stateless_only:
        r, q = v["comm_rows"], o.comm_rows(w)
        for k in q:
            (close if k in ("R", "P") else same)(r[k], q[k], "comm row " + k)
    return v, t


def compare_cumulative(an, o, n_ranks, w_last):
    a, b = an.get_rank_stats(n_ranks), o.rank_stats(n_ranks)
    for k in ("votes", "ops", "bw_cnt"):
        same(a[k], b[k], k)
    close(a["bw_sum"], b["bw_sum"], "bw_sum")
    sa, sb = an.get_verdict(w_last, check=False)["suspects"], o.suspects()
    for k in ("kind", "rank", "votes", "ops"):
        same(sa[k], sb[k], "suspect " + k)
    close(sa["mean_busbw"], sb["mean_busbw"], "suspect mean_busbw")
    return sa


def compare_hang(an, o, w, comm, seq):
    a, b = an.locate_hang(w, comm, seq), o.locate_hang(w, comm, seq)
    assert a["cls"] == b["cls"] and a["n_roots_total"] == b["n_roots"], (a, b)
    for k in ("n_not_entered", "n_hung", "n_not_hung", "n_missing_frames", "stuck_step", "n_members", "min_total"):
        assert a[k] == b[k], (k, a[k], b[k])
    same(a["roots"], b["roots"], "hang roots")
    return a
