"""The five benchmark configurations (plus the single-communicator variant of the fourth) as specs.

Each builder takes size overrides so the tests can run the same structure at a size a CPU
oracle finishes in seconds.
"""
from __future__ import annotations

from typing import List

import torch

from .core import (Family, Fault, Hang, Spec, _py_mix64, OP_ALLREDUCE, OP_ALLGATHER,
                   OP_REDUCESCATTER, OP_SENDRECV)

MiB = 1 << 20


def _pick(seed: int, salt: int, n: int, k: int) -> List[int]:
    """k distinct pseudo-random integers in [0, n)."""
    out: List[int] = []
    i = 0
    while len(out) < k:
        r = _py_mix64((seed << 32) ^ (salt << 16) ^ i) % n
        i += 1
        if r not in out:
            out.append(r)
    return out


def _strided(n_ranks: int, n: int, stride: int) -> torch.Tensor:
    """All groups {base + i*stride, i < n} that tile [0, n_ranks): int64 [n_ranks/n, n]."""
    r = torch.arange(n_ranks, dtype=torch.int64)
    block = n * stride
    first = r[(r % block) < stride]
    return first.unsqueeze(1) + torch.arange(n, dtype=torch.int64).unsqueeze(0) * stride


def cfg1(n_ops: int = 1000) -> Spec:
    fam = Family("ring8", torch.arange(8, dtype=torch.int64).unsqueeze(0), (OP_ALLREDUCE,), 0,
                 bytes_choices=(1 * MiB, 4 * MiB, 16 * MiB, 64 * MiB))
    return Spec("cfg1", 0, 8, [fam], [0], n_ops, 1,
                faults=[Fault(5, "delay_const", 300, 2_000_000)],
                truth={"stragglers": [5], "slow_links": []})


def _three_d(name, seed, tp, pp, dp, pattern, reps, n_windows) -> Spec:
    R = tp * pp * dp
    fam_tp = Family("tp", _strided(R, tp, 1), (OP_ALLREDUCE,), 0)
    fam_pp = Family("pp", _strided(R, pp, tp), (OP_SENDRECV,), fam_tp.members.shape[0])
    fam_dp = Family("dp", _strided(R, dp, tp * pp), (OP_REDUCESCATTER, OP_ALLGATHER),
                    fam_tp.members.shape[0] + fam_pp.members.shape[0])
    return Spec(name, seed, R, [fam_tp, fam_pp, fam_dp], pattern, reps, n_windows)


def cfg2(reps: int = 1000, n_windows: int = 10, tp: int = 8, pp: int = 8, dp: int = 8) -> Spec:
    s = _three_d("cfg2", 1, tp, pp, dp, [0, 1, 2], reps, n_windows)
    nic, strag = _pick(s.seed, 1, s.n_ranks, 2)
    s.faults = [Fault(nic, "bw", factor_milli=400, scope="inter"),
                Fault(strag, "delay_exp", 500, 1_000_000)]
    s.truth = {"stragglers": [strag], "slow_links": [nic]}
    return s


def cfg3(n_rings: int = 16, ring: int = 256, n_done: int = 100, hung_ring: int = 7,
         stuck_pos: int = 1, n_channels: int = 16) -> Spec:
    R = n_rings * ring
    fam = Family("ring", _strided(R, ring, 1), (OP_ALLREDUCE,), 0)
    s = Spec("cfg3", 2, R, [fam], [0], n_done + 1, 1)
    s.hang = Hang(0, hung_ring, 0, n_done, stuck_pos, 23, 24, 64, n_channels)
    s.truth = {"hang_root": [int(fam.members[hung_ring, stuck_pos])], "stuck_step": [23]}
    return s


def cfg4(reps: int = 200, n_windows: int = 100, tp: int = 8, pp: int = 8, dp: int = 64, pattern=(0, 0, 1, 0, 2)) -> Spec:
    """pattern: communicator family of each op slot (0 TP, 1 PP, 2 DP); other patterns single out one kernel path."""
    s = _three_d("cfg4", 3, tp, pp, dp, list(pattern), reps, n_windows)
    r = _pick(s.seed, 1, s.n_ranks, 7)
    s.faults = ([Fault(x, "delay_exp", 200, 500_000) for x in r[:4]]
                + [Fault(x, "bw", factor_milli=500) for x in r[4:6]]
                + [Fault(r[6], "bw", factor_milli=700, scope="intra")])
    s.truth = {"stragglers": sorted(r[:4]), "slow_links": sorted(r[4:7])}
    return s


def cfg4w(reps: int = 1000, n_windows: int = 100, n_ranks: int = 4096) -> Spec:
    fam = Family("world", torch.arange(n_ranks, dtype=torch.int64).unsqueeze(0), (OP_ALLREDUCE,), 0)
    s = Spec("cfg4w", 3, n_ranks, [fam], [0], reps, n_windows)
    r = _pick(s.seed, 1, n_ranks, 6)
    s.faults = ([Fault(x, "delay_exp", 200, 500_000) for x in r[:4]]
                + [Fault(x, "bw", factor_milli=500) for x in r[4:6]])
    s.truth = {"stragglers": sorted(r[:4]), "slow_links": sorted(r[4:6])}
    return s


def cfg5(reps: int = 10, n_windows: int = 50, nodes: int = 2048, mid: int = 128,
         hang_window: int = 25, n_channels: int = 8) -> Spec:
    R = nodes * 8
    ring_n = nodes // 2
    fam_tp = Family("tp", _strided(R, 8, 1), (OP_ALLREDUCE,), 0)
    fam_mid = Family("mid", _strided(R, mid, 1), (OP_ALLGATHER, OP_REDUCESCATTER), R // 8)
    fam_dp = Family("dp", _strided(R, nodes, 8), (OP_ALLREDUCE,), R // 8 + R // mid)
    ring = (torch.arange(ring_n, dtype=torch.int64) * 8 + 3).unsqueeze(0)
    fam_ring = Family("ring", ring, (OP_ALLREDUCE,), R // 8 + R // mid + 8,
                      bytes_choices=(64 * MiB,))
    pattern = [0, 0, 1, 2] * 25 + [3]
    s = Spec("cfg5", 4, R, [fam_tp, fam_mid, fam_dp, fam_ring], pattern, reps, n_windows)
    per_win = reps                       # ring ops per window
    stuck_pos = _py_mix64(s.seed ^ 0xABCD) % ring_n
    s.hang = Hang(3, 0, hang_window, hang_window * per_win + per_win // 2, stuck_pos,
                  41, 42, 64, n_channels)
    r = _pick(s.seed, 1, R, 32)
    s.faults = ([Fault(x, "delay_exp", 200, 500_000) for x in r[:12]]
                + [Fault(x, "bw", factor_milli=500) for x in r[12:22]]
                + [Fault(x, "bw", factor_milli=600, scope="inter") for x in r[22:27]]
                + [Fault(x, "delay_const", 300, 1_000_000) for x in r[27:32]])
    s.truth = {"stragglers": sorted(r[:12] + r[27:32]), "slow_links": sorted(r[12:27]),
               "hang_root": [int(ring[0, stuck_pos])], "stuck_step": [41]}
    return s


PRESETS = {"cfg1": cfg1, "cfg2": cfg2, "cfg3": cfg3, "cfg4": cfg4, "cfg4w": cfg4w, "cfg5": cfg5}
