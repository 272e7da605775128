"""Trace generator core: specs, the counter-based hash, table draws and window synthesis."""
from __future__ import annotations

import json
import os
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import torch

OP_ALLREDUCE, OP_ALLGATHER, OP_REDUCESCATTER, OP_ALLTOALL, OP_SENDRECV, OP_BROADCAST = range(6)

GPUS_PER_NODE = 8
_M64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Python int -> the signed value of its low 64 bits."""
    x &= _M64
    return x - (1 << 64) if x >> 63 else x


_K1 = _s64(0xBF58476D1CE4E5B9)
_K2 = _s64(0x94D049BB133111EB)
_GOLD = _s64(0x9E3779B97F4A7C15)


def _py_mix64(z: int) -> int:
    """splitmix64 output function on a Python int (unsigned 64-bit)."""
    z &= _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    return (z >> s) & ((1 << (64 - s)) - 1)


def mix64(z: torch.Tensor) -> torch.Tensor:
    """splitmix64 output function on an int64 tensor (wrapping arithmetic, logical shifts)."""
    z = (z ^ _lsr(z, 30)) * _K1
    z = (z ^ _lsr(z, 27)) * _K2
    return z ^ _lsr(z, 31)


def draw(seed: int, stream: int, k1: torch.Tensor, k2) -> torch.Tensor:
    """64 hash bits per element, a pure function of (seed, stream, k1, k2)."""
    c = _s64(_py_mix64((seed << 20) ^ stream ^ 0x5EEDC0DE))
    h = mix64(k1 ^ c)
    return mix64(h + k2 * _GOLD)


def hi32(h: torch.Tensor) -> torch.Tensor:
    return _lsr(h, 32)


def lo32(h: torch.Tensor) -> torch.Tensor:
    return h & 0xFFFFFFFF


class _Tables:
    _cache: Dict[str, Dict[str, torch.Tensor]] = {}
    _raw = None

    @classmethod
    def get(cls, device) -> Dict[str, torch.Tensor]:
        key = str(device)
        if key not in cls._cache:
            if cls._raw is None:
                path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "quantile_tables.json")
                with open(path) as f:
                    cls._raw = json.load(f)
                assert cls._raw["n_intervals"] == 4096 and cls._raw["frac_bits"] == 16
            cls._cache[key] = {
                k: torch.tensor(cls._raw[k], dtype=torch.int64, device=device)
                for k in ("normal", "expo", "logn01", "logn10")
            }
        return cls._cache[key]


def table_draw(name: str, u32: torch.Tensor) -> torch.Tensor:
    """Fixed-point (16 fractional bits) quantile of distribution `name` at the 32-bit uniform u32."""
    t = _Tables.get(u32.device)[name]
    idx = u32 >> 20
    frac = u32 & 0xFFFFF
    a = t[idx]
    b = t[idx + 1]
    return a + (((b - a) * frac) >> 20)


# ----------------------------------------------------------------------------------------------
# Specs
# ----------------------------------------------------------------------------------------------
@dataclass
class Family:
    """A set of same-shaped ring communicators (e.g. all TP groups of a job)."""
    name: str
    members: torch.Tensor            # int64 [G, n], ring order, CPU
    ops: Tuple[int, ...]             # op code of seq s is ops[s % len(ops)]
    comm_id0: int                    # communicator id of group g is comm_id0 + g
    bytes_choices: Optional[Tuple[int, ...]] = None   # uniform over these, else lognormal
    bytes_median: int = 32 << 20
    seq0: int = 0


@dataclass
class Fault:
    rank: int
    kind: str                        # 'delay_const' | 'delay_exp' | 'bw'
    prob_milli: int = 1000           # delay faults: fraction of ops hit
    ns: int = 0                      # delay faults: constant or mean delay
    factor_milli: int = 1000         # bw faults: bandwidth multiplier
    scope: str = "all"               # bw faults: 'all' | 'inter' | 'intra' node communicators


@dataclass
class Hang:
    family: int
    group: int
    window: int
    seq: int                         # the op that never completes
    stuck_pos: int                   # ring position of the root rank
    stuck_step: int                  # its Send/Recv counters stop here
    wait_step: int                   # every other member of the ring stalls here
    done_step: int                   # counters of rings that completed the op
    n_channels: int


@dataclass
class Spec:
    name: str
    seed: int
    n_ranks: int
    families: List[Family]
    pattern: List[int]               # family index per op slot, repeated `reps` times per window
    reps: int
    n_windows: int
    faults: List[Fault] = field(default_factory=list)
    hang: Optional[Hang] = None
    t0_ns: int = 1_000_000_000
    spacing_ns: int = 5_000_000
    jitter_ns: int = 20_000
    truth: Dict[str, List[int]] = field(default_factory=dict)

    @property
    def ops_per_window(self) -> int:
        return len(self.pattern) * self.reps


@dataclass
class Window:
    window_id: int
    cols: Dict[str, torch.Tensor]
    now_ns: int
    frames: Optional[Dict[str, torch.Tensor]] = None
    n_channels: int = 0

    @property
    def n_rec(self) -> int:
        return int(self.cols["rank"].numel())


def registry(spec: Spec) -> List[Tuple[int, List[int], int]]:
    """(communicator id, member ranks in ring order, first sequence number) for every communicator."""
    out = []
    for fam in spec.families:
        for g in range(fam.members.shape[0]):
            out.append((fam.comm_id0 + g, [int(x) for x in fam.members[g]], fam.seq0))
    return out


def _family_tables(spec: Spec, device):
    R = spec.n_ranks
    F = len(spec.families)
    grp = torch.full((F, R), -1, dtype=torch.int64)
    intra = []
    for f, fam in enumerate(spec.families):
        G, n = fam.members.shape
        g_idx = torch.arange(G).unsqueeze(1).expand(G, n)
        grp[f, fam.members.reshape(-1)] = g_idx.reshape(-1)
        node = fam.members // GPUS_PER_NODE
        intra.append((node == node[:, :1]).all(dim=1))
    return grp.to(device), [t.to(device) for t in intra]


def records_per_window(spec: Spec) -> int:
    """Record count of a window that no hang truncates."""
    grp, _ = _family_tables(spec, "cpu")
    per_fam = (grp >= 0).sum(dim=1)
    cnt = [spec.pattern.count(f) for f in range(len(spec.families))]
    return int(sum(int(per_fam[f]) * cnt[f] for f in range(len(spec.families))) * spec.reps)


def gen_window(spec: Spec, w: int, device="cpu", order: str = "rank_major") -> Window:
    """Synthesize window `w` of `spec` on `device`.

    order: 'rank_major' (each rank's batch contiguous, ops in program order), 'arrival' (sorted by
    exit time, in-flight records last) or 'shuffled'.
    """
    dev = torch.device(device)
    R, L, O = spec.n_ranks, len(spec.pattern), spec.ops_per_window
    F = len(spec.families)
    seed = spec.seed
    grp, intra = _family_tables(spec, dev)

    pat = torch.tensor(spec.pattern, dtype=torch.int64, device=dev)
    cnt = torch.tensor([spec.pattern.count(f) for f in range(F)], dtype=torch.int64, device=dev)
    occ = torch.tensor([spec.pattern[:i].count(spec.pattern[i]) for i in range(L)],
                       dtype=torch.int64, device=dev)
    seq0 = torch.tensor([fam.seq0 for fam in spec.families], dtype=torch.int64, device=dev)
    cid0 = torch.tensor([fam.comm_id0 for fam in spec.families], dtype=torch.int64, device=dev)

    o = torch.arange(O, dtype=torch.int64, device=dev)
    og = w * O + o                                   # op slot in the rank's whole program
    fam_o = pat[o % L]                               # [O]
    seq_o = (og // L) * cnt[fam_o] + occ[o % L] + seq0[fam_o]

    g = grp[fam_o].t().contiguous()                  # [R, O] group index or -1
    valid = g >= 0
    rank = torch.arange(R, dtype=torch.int64, device=dev).unsqueeze(1).expand(R, O)
    comm = cid0[fam_o].unsqueeze(0) + g
    seq = seq_o.unsqueeze(0).expand(R, O)
    key = (comm << 32) | seq                         # one key per (communicator, op)

    # op type, bytes and locality: shared by all members of a (communicator, op)
    op = torch.zeros((R, O), dtype=torch.int64, device=dev)
    nbytes = torch.zeros((R, O), dtype=torch.int64, device=dev)
    is_intra = torch.zeros((R, O), dtype=torch.bool, device=dev)
    hb = draw(seed, 1, key, 0)
    for f, fam in enumerate(spec.families):
        cols = (fam_o == f).nonzero().flatten()
        if cols.numel() == 0:
            continue
        ops_t = torch.tensor(fam.ops, dtype=torch.int64, device=dev)
        op[:, cols] = ops_t[seq_o[cols] % len(fam.ops)].unsqueeze(0).expand(R, -1)
        h = hb[:, cols]
        if fam.bytes_choices is not None:
            ch = torch.tensor(fam.bytes_choices, dtype=torch.int64, device=dev)
            b = ch[hi32(h) % len(fam.bytes_choices)]
        else:
            b = (fam.bytes_median * table_draw("logn10", hi32(h))) >> 16
            b = b.clamp(4 << 10, 4 << 30) & ~3
        nbytes[:, cols] = b
        gi = g[:, cols].clamp(min=0)
        is_intra[:, cols] = intra[f][gi]

    # per-rank fault tables
    d_prob = torch.zeros(R, dtype=torch.int64)
    d_ns = torch.zeros(R, dtype=torch.int64)
    d_exp = torch.zeros(R, dtype=torch.bool)
    bw = {s: torch.full((R,), 1000, dtype=torch.int64) for s in ("all", "inter", "intra")}
    for ft in spec.faults:
        if ft.kind in ("delay_const", "delay_exp"):
            d_prob[ft.rank], d_ns[ft.rank], d_exp[ft.rank] = ft.prob_milli, ft.ns, ft.kind == "delay_exp"
        elif ft.kind == "bw":
            bw[ft.scope][ft.rank] = ft.factor_milli
        else:
            raise ValueError(ft.kind)
    d_prob, d_ns, d_exp = d_prob.to(dev), d_ns.to(dev), d_exp.to(dev)
    bw = {s: t.to(dev) for s, t in bw.items()}

    # enter time = base + jitter + injected delay
    jit = (table_draw("normal", hi32(draw(seed, 2, key, rank))) * spec.jitter_ns) >> 16
    hd = draw(seed, 3, key, rank)
    hit = (hi32(hd) % 1000) < d_prob.unsqueeze(1)
    dly_exp = (table_draw("expo", lo32(hd)) * d_ns.unsqueeze(1)) >> 16
    dly = torch.where(d_exp.unsqueeze(1), dly_exp, d_ns.unsqueeze(1).expand(R, O))
    dly = torch.where(hit, dly, torch.zeros_like(dly))
    t_enter = spec.t0_ns + og.unsqueeze(0) * spec.spacing_ns + jit + dly

    # duration: lognormal around 2 ms per 16 MiB, stretched by the rank's bandwidth factors
    med = (nbytes * 2_000_000) >> 24
    dur = (med * table_draw("logn01", hi32(draw(seed, 4, key, rank)))) >> 16
    dur = (dur * 1000) // bw["all"].unsqueeze(1)
    scoped = torch.where(is_intra, bw["intra"].unsqueeze(1), bw["inter"].unsqueeze(1))
    dur = ((dur * 1000) // scoped).clamp(min=1)
    t_exit = t_enter + dur
    chg = ((dur + 999_999) // 1_000_000).clamp(min=1)

    frames = None
    n_channels = 0
    hg = spec.hang
    if hg is not None and w >= hg.window:
        in_ring = (fam_o == hg.family).unsqueeze(0) & (g == hg.group)
        valid = valid & ~(in_ring & (seq > hg.seq))
        stuck = in_ring & (seq == hg.seq)
        t_exit = torch.where(stuck, torch.full_like(t_exit, -1), t_exit)
        chg = torch.where(stuck, torch.zeros_like(chg), chg)
    if hg is not None and w == hg.window:
        fam = spec.families[hg.family]
        G, n = fam.members.shape
        C = hg.n_channels
        n_channels = C
        prog = torch.full((G, n, C, 2), hg.done_step, dtype=torch.int64)
        prog[hg.group] = hg.wait_step
        prog[hg.group, hg.stuck_pos] = hg.stuck_step
        frames = {
            "f_rank": fam.members.reshape(-1).to(torch.int32).to(dev),
            "f_comm": (fam.comm_id0 + torch.arange(G).unsqueeze(1).expand(G, n)).reshape(-1).to(torch.int32).to(dev),
            "f_seq": torch.full((G * n,), hg.seq, dtype=torch.int32, device=dev),
            "progress": prog.reshape(G * n, C, 2).to(torch.int32).to(dev).contiguous(),
        }

    def flat(t):
        return t.reshape(-1)[valid.reshape(-1)] if t.shape == valid.shape else t.expand(R, O).reshape(-1)[valid.reshape(-1)]

    cols = {
        "rank": flat(rank), "comm": flat(comm), "seq": flat(seq), "op": flat(op),
        "bytes": flat(nbytes), "t_enter": flat(t_enter), "t_exit": flat(t_exit),
        "send_chg": flat(chg), "recv_chg": flat(chg),
    }
    n_rec = cols["rank"].numel()
    if order != "rank_major":
        idx = torch.arange(n_rec, dtype=torch.int64, device=dev)
        if order == "arrival":
            k = torch.where(cols["t_exit"] < 0, torch.full_like(cols["t_exit"], (1 << 63) - 1), cols["t_exit"])
            perm = torch.sort(k, stable=True).indices
        elif order == "shuffled":
            perm = torch.sort(_lsr(draw(seed, 9, idx + (w << 40), 0), 1), stable=True).indices
        else:
            raise ValueError(order)
        cols = {k_: v[perm] for k_, v in cols.items()}
    out = {
        "rank": cols["rank"].to(torch.int32), "comm": cols["comm"].to(torch.int32),
        "seq": cols["seq"].to(torch.int32), "op": cols["op"].to(torch.uint8),
        "bytes": cols["bytes"].contiguous(), "t_enter": cols["t_enter"].contiguous(),
        "t_exit": cols["t_exit"].contiguous(),
        "send_chg": cols["send_chg"].to(torch.int32), "recv_chg": cols["recv_chg"].to(torch.int32),
    }
    out = {k_: v.contiguous() for k_, v in out.items()}
    now = spec.t0_ns + ((w + 1) * O) * spec.spacing_ns + (600_000_000_000 if hg is not None else 1_000_000_000)
    return Window(window_id=w, cols=out, now_ns=int(now), frames=frames, n_channels=n_channels)
