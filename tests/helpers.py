"""Hand-built traces for the tests: plain Python lists -> SoA numpy columns."""
import numpy as np

MiB = 1 << 20
ALLREDUCE, ALLGATHER, REDUCESCATTER, ALLTOALL, SENDRECV, BROADCAST = range(6)


def make_cols(records, with_rates=True):
    """records: iterable of dicts with keys rank, comm, seq, t_enter, t_exit and optionally
    op (default allreduce), bytes (default 16 MiB), send_chg, recv_chg (default 1)."""
    records = list(records)
    g = lambda k, d: [r.get(k, d) for r in records]
    cols = {
        "rank": np.array(g("rank", 0), dtype=np.uint32),
        "comm": np.array(g("comm", 0), dtype=np.uint32),
        "seq": np.array(g("seq", 0), dtype=np.uint32),
        "op": np.array(g("op", ALLREDUCE), dtype=np.uint8),
        "bytes": np.array(g("bytes", 16 * MiB), dtype=np.uint64),
        "t_enter": np.array(g("t_enter", 0), dtype=np.int64),
        "t_exit": np.array(g("t_exit", 0), dtype=np.int64),
    }
    if with_rates:
        cols["send_chg"] = np.array(g("send_chg", 1), dtype=np.uint32)
        cols["recv_chg"] = np.array(g("recv_chg", 1), dtype=np.uint32)
    return cols


def group_trace(durs_per_seq, enters_per_seq=None, comm=0, ranks=None, seq0=0, t0=1_000_000_000, spacing=50_000_000, **kw):
    """One record per (seq, member): durations durs_per_seq[s][i], enter offsets enters_per_seq[s][i]."""
    recs = []
    for s, durs in enumerate(durs_per_seq):
        n = len(durs)
        rk = ranks if ranks is not None else list(range(n))
        for i in range(n):
            te = t0 + s * spacing + (enters_per_seq[s][i] if enters_per_seq is not None else 0)
            recs.append(dict(rank=rk[i], comm=comm, seq=seq0 + s, t_enter=te, t_exit=te + durs[i], **kw))
    return recs


def frames_from(entries, n_channels):
    """entries: list of (rank, comm, seq, [(send, recv)] * n_channels)."""
    return {
        "f_rank": np.array([e[0] for e in entries], dtype=np.uint32),
        "f_comm": np.array([e[1] for e in entries], dtype=np.uint32),
        "f_seq": np.array([e[2] for e in entries], dtype=np.uint32),
        "progress": np.array([e[3] for e in entries], dtype=np.uint32).reshape(len(entries), n_channels, 2),
    }
