"""ccld_derive_rates against the oracle: counter changes per op from raw probe samples (Sec. 4.1.2)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
import oracle as orc
import paper_2605_04478_b200 as ccld
import tracegen as tg

pytestmark = pytest.mark.gpu
MS = 1_000_000


def _check(an, rank, te, tx, off, tn, sc, rc):
    dev = "cuda"
    t = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a).astype(dt)).to(dev)
    s, r = an.derive_rates(t(rank, np.int32), t(te, np.int64), t(tx, np.int64), t(off, np.int64), t(tn, np.int64),
                           t(sc, np.int32), t(rc, np.int32))
    torch.cuda.synchronize()
    es, er = orc.derive_rates(rank, te, tx, off, tn, sc, rc)
    assert np.array_equal(s.cpu().numpy().view(np.uint32), es)
    assert np.array_equal(r.cpu().numpy().view(np.uint32), er)
    return es, er


def test_random_series_ragged_tiles_empty_ranks_in_flight_ops():
    """Several tick tiles with a ragged tail, ranks of 0, 1, 2 and thousands of ticks (segments that start inside a
    thread's run and inside a tile), records in flight, before the first and after the last tick, an unknown rank."""
    rng = np.random.default_rng(21)
    sizes = [0, 1, 2, 0, 3000, 7, 0, 0, 2049, 5000, 1, 0]
    series_t, series_s, series_r = [], [], []
    for n in sizes:
        series_t.append(np.sort(rng.choice(20_000 * MS, size=n, replace=False)))
        series_s.append(np.cumsum(rng.integers(0, 3, n)))
        series_r.append(np.cumsum(rng.integers(0, 2, n)))
    off = np.cumsum([0] + sizes)
    tn = np.concatenate(series_t); sc = np.concatenate(series_s); rc = np.concatenate(series_r)
    n_rec = 5000
    rank = rng.integers(0, len(sizes) + 1, n_rec)                                  # includes one id beyond the table
    te = rng.integers(-5 * MS, 20_000 * MS, n_rec); tx = te + rng.integers(0, 500 * MS, n_rec)
    tx[rng.random(n_rec) < 0.05] = -1
    tx[:10] = te[:10]                                                              # zero-length ops
    an = ccld.Analyzer()
    es, _ = _check(an, rank, te, tx, off, tn, sc, rc)
    assert es.max() > 50
    # counters that wrap around 2^32 still compare tick to tick
    sc2 = (sc.astype(np.uint64) * 7_000_003 % (1 << 32)).astype(np.uint32)
    _check(an, rank, te, tx, off, tn, sc2.view(np.int32), rc)


def test_paper_example_and_pipeline_input():
    """The 2-changes against 7-changes example of Sec. 4.1.2, then samples generated for a window of a 3D-parallel job:
    the derived columns equal the oracle's and are accepted by the analyzer as its rate columns."""
    normal = [min(8, 4 * k) for k in range(11)]; slow = [0, 1, 2, 3, 4, 6, 7, 8, 8, 8, 8]
    tn = np.tile(np.arange(11) * MS, 2)
    an = ccld.Analyzer()
    es, _ = _check(an, [0, 1], [0, 0], [10 * MS, 10 * MS], [0, 11, 22], tn, np.array(normal + slow), np.zeros(22))
    assert list(es) == [2, 7]

    spec = tg.cfg2(reps=40, n_windows=1, tp=8, pp=2, dp=4)
    win = tg.gen_window(spec, 0, device="cuda")
    ticks = tg.gen_ticks(win.cols, spec.n_ranks)
    s, r = an.derive_rates(win.cols["rank"], win.cols["t_enter"], win.cols["t_exit"], ticks["tick_off"], ticks["tick_ns"],
                           ticks["send_count"], ticks["recv_count"])
    torch.cuda.synchronize()
    c = {k: v.cpu().numpy() for k, v in win.cols.items()}
    k = {k: v.cpu().numpy() for k, v in ticks.items()}
    es, er = orc.derive_rates(c["rank"], c["t_enter"], c["t_exit"], k["tick_off"], k["tick_ns"], k["send_count"], k["recv_count"])
    assert np.array_equal(s.cpu().numpy().view(np.uint32), es) and np.array_equal(r.cpu().numpy().view(np.uint32), er)
    assert 1 <= np.median(es) <= 8                              # ops of a few ms sampled every 1 ms
    cols = dict(win.cols); cols["send_chg"] = s; cols["recv_chg"] = r
    o = orc.Oracle()
    for cid, ranks, seq0 in tg.registry(spec):
        an.comm_register(cid, ranks, 0, seq0); o.comm_register(cid, ranks, seq0)
    an.trace_upload(0, cols); o.upload(0, cols)
    an.analyze_window(0, 1, win.now_ns); o.analyze(0, 1, win.now_ns)
    t, g = an.get_optable(0), o.groups(0)
    assert np.array_equal(t["max_chg"], g["max_chg"]) and np.array_equal(t["rank_max_chg"], g["rank_max_chg"])


def _series(rng, n_ranks, n_ticks, period_ms=1):
    off = np.arange(n_ranks + 1) * n_ticks
    tn = np.concatenate([np.arange(n_ticks) * period_ms * MS + rng.integers(0, MS) for _ in range(n_ranks)])
    sc = np.concatenate([np.cumsum(rng.integers(0, 2, n_ticks)) for _ in range(n_ranks)])
    rc = np.concatenate([np.cumsum(rng.integers(0, 3, n_ticks) // 2) for _ in range(n_ranks)])
    return off, tn, sc, rc


def test_ops_of_29_to_36_ticks_at_every_place_in_the_table():
    """Ops that span 29 to 36 ticks (around a warp's width), from before a rank's first tick, after it, in the middle of
    its ticks, up to its last tick and in flight with as many ticks left, each ending on a tick and between two."""
    rng = np.random.default_rng(3)
    off, tn, sc, rc = _series(rng, 3, 200)
    rank, te, tx = [], [], []
    for r in range(3):
        t = tn[off[r]:off[r + 1]]
        for span in range(29, 37):
            for first in (0, 1, 57, 200 - span):                    # from before the first tick, after it, mid-table, to the last tick
                a = t[first] - 1 if first else t[0] - 5
                rank.append(r); te.append(a); tx.append(t[first + span - 1])           # `span` ticks in (a, b]
                rank.append(r); te.append(a); tx.append(t[first + span - 1] + MS // 2)
            rank.append(r); te.append(t[200 - span] - 1); tx.append(-1)                 # in flight, `span` ticks left
    _check(ccld.Analyzer(), np.array(rank), np.array(te), np.array(tx), off, tn, sc, rc)


def test_a_few_long_ops_among_short_ones():
    """Thousands of ops of a few ticks and ten that span hundreds to thousands of ticks (two of them in flight)."""
    rng = np.random.default_rng(4)
    off, tn, sc, rc = _series(rng, 4, 20_000)
    n = 3000
    rank = rng.integers(0, 4, n); te = rng.integers(0, 19_900 * MS, n); tx = te + rng.integers(0, 6 * MS, n)
    long_ = rng.choice(n, 10, replace=False)
    tx[long_] = te[long_] + rng.integers(100 * MS, 9_000 * MS, 10)
    tx[long_[:2]] = -1
    es, _ = _check(ccld.Analyzer(), rank, te, tx, off, tn, sc, rc)
    assert es[long_].min() > 20 and np.median(es) <= 4


def test_every_op_spans_hundreds_of_ticks():
    """Every op spans 200 to 300 of its rank's 400 ticks, a tenth of them in flight."""
    rng = np.random.default_rng(5)
    off, tn, sc, rc = _series(rng, 50, 400)
    n = 3000
    rank = rng.integers(0, 50, n); te = rng.integers(-10 * MS, 150 * MS, n); tx = te + rng.integers(200 * MS, 300 * MS, n)
    tx[rng.random(n) < 0.1] = -1
    es, _ = _check(ccld.Analyzer(), rank, te, tx, off, tn, sc, rc)
    assert np.median(es) > 50
