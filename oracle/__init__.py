"""ctypes front end of the CPU oracle (`ccld_oracle.cpp`). TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package;
the product path (the CUDA library and its Python binding) never does.
"""
from __future__ import annotations

import ctypes as C
from typing import Dict, Optional

import numpy as np

from .build import build as build_oracle

PARAM_ORDER = ("tbase_init_ns", "theta_slow_milli", "alpha_milli", "beta_milli", "m_max_rounds",
               "m_max_ns", "hang_ns", "barrier_bytes", "slow_rep_threshold", "k_milli", "min_group",
               "vote_rep_milli")

# Defaults quoted by the paper: theta_slow ~ 3 (Sec. 4.2.1), alpha = 0.4 and beta = 0.6 (Sec. 4.2.2),
# m = min(100 rounds, rounds of the first two minutes) (Sec. 4.2.1), hang threshold 5 min (Sec. 6.1),
# barrier = AllReduce of fewer than 4 bytes (Sec. 4.2.1). The rest are this repository's choices.
DEFAULT_PARAMS = dict(tbase_init_ns=2_000_000, theta_slow_milli=3000, alpha_milli=400, beta_milli=600,
                      m_max_rounds=100, m_max_ns=120_000_000_000, hang_ns=300_000_000_000,
                      barrier_bytes=4, slow_rep_threshold=1, k_milli=5189, min_group=4,
                      vote_rep_milli=100)

GROUP_I64 = ("e_min", "arrival_skew", "t_max", "t_min", "span", "med_skew", "mad_skew", "med_dur", "mad_dur")
GROUP_U32 = ("rank_tmin", "rank_tmax", "max_chg", "rank_max_chg", "n_present", "gflags")
COMM_U32 = ("comm", "n_rounds", "sel_seq", "cls", "slow_detected", "located", "baseline_static",
            "rate_source", "root_comp", "root_comm")
SIZES = ("n_records", "n_groups", "n_slots", "n_comm_rows", "n_alerts", "n_rejected", "n_complete",
         "n_incomplete", "n_barrier", "n_analysed", "n_flag_skew", "n_flag_dur", "n_opset_mismatch", "error_bits")

_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build_oracle())
        _lib.orc_create.restype = C.c_void_p
        _lib.orc_create.argtypes = [C.c_void_p, C.c_int]
        _lib.orc_destroy.argtypes = [C.c_void_p]
        for name in ("orc_comm_register", "orc_upload", "orc_release", "orc_analyze", "orc_window_sizes",
                     "orc_copy_groups", "orc_copy_slots", "orc_copy_comm_rows", "orc_copy_alerts",
                     "orc_copy_rank_stats", "orc_add_rank_stats", "orc_suspects", "orc_locate_hang", "orc_attach_opset", "orc_opset_check", "orc_comm_set_layers"):
            getattr(_lib, name).restype = C.c_int
        _lib.orc_derive_rates.restype = None
    return _lib


def _np(x, dtype):
    if x is None:
        return None
    if hasattr(x, "detach"):
        x = x.detach().cpu().numpy()
    a = np.ascontiguousarray(x)
    if a.dtype != np.dtype(dtype):
        a = a.view(dtype) if a.dtype.itemsize == np.dtype(dtype).itemsize else a.astype(dtype)
    return a


def _p(a):
    return None if a is None else C.c_void_p(a.ctypes.data)


class Oracle:
    def __init__(self, params: Optional[Dict[str, int]] = None):
        self.lib = _load()
        self.params = dict(DEFAULT_PARAMS)
        if params:
            self.params.update(params)
        pv = np.array([self.params[k] for k in PARAM_ORDER], dtype=np.int64)
        self.h = C.c_void_p(self.lib.orc_create(_p(pv), len(pv)))
        assert self.h.value

    def __del__(self):
        if getattr(self, "h", None) is not None and self.h.value:
            self.lib.orc_destroy(self.h)
            self.h = None

    def comm_register(self, comm: int, ranks, seq0: int = 0) -> int:
        r = _np(np.asarray(ranks), np.uint32)
        return self.lib.orc_comm_register(self.h, C.c_uint32(comm), _p(r), C.c_uint32(len(r)), C.c_uint32(seq0))

    def comm_set_layers(self, comm: int, layers) -> int:
        a = _np(layers, np.uint32)
        return self.lib.orc_comm_set_layers(self.h, C.c_uint32(comm), _p(a))

    def upload(self, window_id: int, cols, frames=None, n_channels: int = 0) -> int:
        a = {
            "rank": _np(cols["rank"], np.uint32), "comm": _np(cols["comm"], np.uint32), "seq": _np(cols["seq"], np.uint32),
            "op": _np(cols["op"], np.uint8), "bytes": _np(cols["bytes"], np.uint64),
            "t_enter": _np(cols["t_enter"], np.int64), "t_exit": _np(cols["t_exit"], np.int64),
            "send_chg": _np(cols.get("send_chg"), np.uint32), "recv_chg": _np(cols.get("recv_chg"), np.uint32),
        }
        n = len(a["rank"])
        nf = 0
        fr = fc = fs = pr = None
        if frames is not None:
            fr, fc, fs = (_np(frames[k], np.uint32) for k in ("f_rank", "f_comm", "f_seq"))
            pr = _np(frames["progress"], np.uint32)
            nf = len(fr)
        return self.lib.orc_upload(self.h, C.c_uint32(window_id), C.c_uint64(n), _p(a["rank"]), _p(a["comm"]), _p(a["seq"]),
                                   _p(a["op"]), _p(a["bytes"]), _p(a["t_enter"]), _p(a["t_exit"]), _p(a["send_chg"]),
                                   _p(a["recv_chg"]), C.c_uint32(nf), _p(fr), _p(fc), _p(fs), C.c_uint32(n_channels), _p(pr))

    def release(self, window_id: int) -> int:
        return self.lib.orc_release(self.h, C.c_uint32(window_id))

    def analyze(self, first_window: int, n_windows: int, now_ns: int) -> int:
        return self.lib.orc_analyze(self.h, C.c_uint32(first_window), C.c_uint32(n_windows), C.c_int64(now_ns))

    def sizes(self, window_id: int) -> Dict[str, int]:
        s = np.zeros(14, dtype=np.uint64)
        rc = self.lib.orc_window_sizes(self.h, C.c_uint32(window_id), _p(s))
        assert rc == 0
        return {k: int(v) for k, v in zip(SIZES, s)}

    def groups(self, window_id: int) -> Dict[str, np.ndarray]:
        G = self.sizes(window_id)["n_groups"]
        comm = np.zeros(G, np.uint32); seq = np.zeros(G, np.uint32); slot0 = np.zeros(G, np.uint64)
        i9 = np.zeros((9, G), np.int64); u6 = np.zeros((6, G), np.uint32); bw = np.zeros(G, np.float64)
        self.lib.orc_copy_groups(self.h, C.c_uint32(window_id), _p(comm), _p(seq), _p(slot0), _p(i9), _p(u6), _p(bw))
        out = {"comm": comm, "seq": seq, "slot0": slot0, "busbw": bw}
        out.update({k: i9[i] for i, k in enumerate(GROUP_I64)})
        out.update({k: u6[i] for i, k in enumerate(GROUP_U32)})
        return out

    def slots(self, window_id: int):
        S = self.sizes(window_id)["n_slots"]
        flags = np.zeros(S, np.uint8); perm = np.zeros(S, np.uint32)
        self.lib.orc_copy_slots(self.h, C.c_uint32(window_id), _p(flags), _p(perm))
        return flags, perm

    def comm_rows(self, window_id: int) -> Dict[str, np.ndarray]:
        n = self.sizes(window_id)["n_comm_rows"]
        u10 = np.zeros((10, n), np.uint32); u3 = np.zeros((3, n), np.uint64); i3 = np.zeros((3, n), np.int64); f2 = np.zeros((2, n), np.float64)
        self.lib.orc_copy_comm_rows(self.h, C.c_uint32(window_id), _p(u10), _p(u3), _p(i3), _p(f2))
        out = {k: u10[i] for i, k in enumerate(COMM_U32)}
        out.update(slow_count=u3[0], rounds_total=u3[1], m=u3[2], t_max=i3[0], t_min=i3[1], t_base=i3[2], R=f2[0], P=f2[1])
        return out

    def alerts(self, window_id: int) -> Dict[str, np.ndarray]:
        n = self.sizes(window_id)["n_alerts"]
        comm = np.zeros(n, np.uint32); seq = np.zeros(n, np.uint32); age = np.zeros(n, np.int64)
        self.lib.orc_copy_alerts(self.h, C.c_uint32(window_id), _p(comm), _p(seq), _p(age))
        return {"comm": comm, "seq": seq, "age_ns": age}

    def rank_stats(self, n_ranks: int) -> Dict[str, np.ndarray]:
        votes = np.zeros((n_ranks, 4), np.uint32); ops = np.zeros(n_ranks, np.uint32)
        cnt = np.zeros(n_ranks, np.uint32); bw = np.zeros(n_ranks, np.float64)
        self.lib.orc_copy_rank_stats(self.h, C.c_uint32(n_ranks), _p(votes), _p(ops), _p(cnt), _p(bw))
        return {"votes": votes, "ops": ops, "bw_cnt": cnt, "bw_sum": bw}

    def add_rank_stats(self, st: Dict[str, np.ndarray]) -> int:
        """Adds the per-rank statistics another instance returned from rank_stats() to this instance's."""
        v = _np(st["votes"], np.uint32); ops = _np(st["ops"], np.uint32); cnt = _np(st["bw_cnt"], np.uint32); bw = _np(st["bw_sum"], np.float64)
        return self.lib.orc_add_rank_stats(self.h, C.c_uint32(len(ops)), _p(v), _p(ops), _p(cnt), _p(bw))

    def suspects(self, cap: int = 65536) -> Dict[str, np.ndarray]:
        kind = np.zeros(cap, np.uint32); rank = np.zeros(cap, np.uint32); votes = np.zeros(cap, np.uint32)
        ops = np.zeros(cap, np.uint32); bw = np.zeros(cap, np.float64)
        n = self.lib.orc_suspects(self.h, C.c_uint32(cap), _p(kind), _p(rank), _p(votes), _p(ops), _p(bw))
        m = min(n, cap)
        return {"n_total": n, "kind": kind[:m], "rank": rank[:m], "votes": votes[:m], "ops": ops[:m], "mean_busbw": bw[:m]}

    def attach_opset(self, window_id: int, algo, proto) -> int:
        a = _np(algo, np.uint8); b = _np(proto, np.uint8)
        return self.lib.orc_attach_opset(self.h, C.c_uint32(window_id), _p(a), _p(b))

    def opset_check(self, window_id: int, comm: int, seq: int, cap: int = 65536) -> Dict[str, object]:
        out = np.zeros(7, np.uint32); by = np.zeros(1, np.uint64); ranks = np.zeros(cap, np.uint32)
        rc = self.lib.orc_opset_check(self.h, C.c_uint32(window_id), C.c_uint32(comm), C.c_uint32(seq), _p(out), _p(by), C.c_uint32(cap), _p(ranks))
        assert rc == 0
        d = {k: int(v) for k, v in zip(("n_members", "n_present", "n_deviating_total", "majority_count", "op", "algo", "proto"), out)}
        d["bytes"] = int(by[0])
        d["ranks"] = ranks[:min(d["n_deviating_total"], cap)].copy()
        return d

    def locate_hang(self, window_id: int, comm: int, seq: int, cap: int = 65536) -> Dict[str, object]:
        out = np.zeros(8, np.uint32); mn = np.zeros(1, np.uint64); roots = np.zeros(cap, np.uint32)
        rc = self.lib.orc_locate_hang(self.h, C.c_uint32(window_id), C.c_uint32(comm), C.c_uint32(seq), _p(out), _p(mn),
                                      C.c_uint32(cap), _p(roots))
        assert rc == 0
        keys = ("cls", "n_roots", "n_not_entered", "n_hung", "n_not_hung", "n_missing_frames", "stuck_step", "n_members")
        d = {k: int(v) for k, v in zip(keys, out)}
        d["min_total"] = int(mn[0])
        d["roots"] = roots[:min(d["n_roots"], cap)].copy()
        return d


def derive_rates(rank, t_enter, t_exit, tick_off, tick_ns, send_count, recv_count):
    """Counter changes per record from raw probe samples (Sec. 4.1.2); returns (send_chg, recv_chg) as uint32 arrays."""
    lib = _load()
    rank = _np(rank, np.uint32); te = _np(t_enter, np.int64); tx = _np(t_exit, np.int64)
    off = _np(tick_off, np.uint64); tn = _np(tick_ns, np.int64); sc = _np(send_count, np.uint32); rc = _np(recv_count, np.uint32)
    n = len(rank)
    out_s = np.zeros(n, np.uint32); out_r = np.zeros(n, np.uint32)
    lib.orc_derive_rates(C.c_uint64(n), _p(rank), _p(te), _p(tx), C.c_uint32(len(off) - 1), _p(off), _p(tn), _p(sc), _p(rc),
                         _p(out_s), _p(out_r))
    return out_s, out_r


def analyze_windows_independently(registry, windows, n_ranks: int, threads: int = 1, params=None, keep=None):
    """Each window on a fresh Oracle of its own (one instance per thread at a time; ctypes calls release the GIL, so
    `threads` host cores work side by side). `windows` yields (window_id, cols, now_ns) with CPU columns. Returns the
    summed per-rank statistics, the per-window size dictionaries and the number of records analysed. Per-window results
    that depend on earlier windows (the Eq. 1 baseline, the repetition counter) are not meaningful here; the per-op
    table, flags, counts and the per-rank sums are. keep(window_id, oracle) is called before an instance is dropped.
    """
    from concurrent.futures import ThreadPoolExecutor

    def one(item):
        wid, cols, now = item
        o = Oracle(params)
        for cid, ranks, seq0 in registry:
            o.comm_register(cid, ranks, seq0)
        o.upload(wid, cols)
        o.analyze(wid, 1, now)
        sz = o.sizes(wid)
        st = o.rank_stats(n_ranks)
        if keep is not None:
            keep(wid, o)
        return wid, sz, st

    total = {"votes": np.zeros((n_ranks, 4), np.uint32), "ops": np.zeros(n_ranks, np.uint32),
             "bw_cnt": np.zeros(n_ranks, np.uint32), "bw_sum": np.zeros(n_ranks, np.float64)}
    sizes, n_rec = {}, 0
    with ThreadPoolExecutor(max_workers=max(1, threads)) as ex:
        # windows are pulled lazily, at most 2 x threads in flight, so host memory stays bounded
        import itertools
        it = iter(windows)
        pending = [ex.submit(one, item) for item in itertools.islice(it, 2 * max(1, threads))]
        while pending:
            wid, sz, st = pending.pop(0).result()
            for k in total:
                total[k] += st[k]
            sizes[wid] = sz
            n_rec += sz["n_records"]
            nxt = next(it, None)
            if nxt is not None:
                pending.append(ex.submit(one, nxt))
    return total, sizes, n_rec
