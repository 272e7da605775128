"""Seeded raw probe samples (SendCount / RecvCount per sampling tick) that go with a window of trace records.

Input generation only: what a rank probe sampling its counters every `period_ns` would have seen while the window's
ops ran. Each op advances the rank's counters by `steps` sends and receives, spread evenly over the op's duration; an
op in flight stops half way. Integer arithmetic on torch tensors: the same bits on the CPU and on a GPU.
"""
from typing import Dict

import torch

from .core import draw


def gen_ticks(cols: Dict[str, torch.Tensor], n_ranks: int, period_ns: int = 1_000_000, steps: int = 8, seed: int = 0) -> Dict[str, torch.Tensor]:
    """Returns tick_off int64 [n_ranks + 1], tick_ns int64, send_count int32, recv_count int32 (all ranks share one grid
    length; every rank's grid has its own phase)."""
    rank = cols["rank"].to(torch.int64); te = cols["t_enter"]; tx = cols["t_exit"]
    dev = rank.device
    done = tx >= 0
    t_lo = int(te.min()) - period_ns
    t_hi = int(torch.where(done, tx, te).max()) + 2 * period_ns
    T = (t_hi - t_lo) // period_ns + 1
    assert t_hi < (1 << 44) and n_ranks < (1 << 19)
    r_ids = torch.arange(n_ranks, device=dev, dtype=torch.int64)
    phase = (draw(seed, 900, r_ids, 0) & 0x7FFFFFFF) % period_ns
    tick = t_lo + phase[:, None] + torch.arange(T, device=dev, dtype=torch.int64)[None, :] * period_ns      # [n_ranks, T]
    # records in (rank, enter time) order, and where each rank's records start
    key = (rank << 44) + te
    order = torch.argsort(key)
    key_s = key[order]; te_s = te[order]; tx_s = tx[order]
    seg = torch.searchsorted(key_s, r_ids << 44)                                   # first record of each rank
    j = torch.searchsorted(key_s, ((r_ids[:, None] << 44) + tick).reshape(-1), right=True).reshape(n_ranks, T) - seg[:, None]
    # ops entered by the tick: all but the last count as complete, the last one by its progress
    last = (seg[:, None] + j - 1).clamp(min=0, max=max(int(key_s.numel()) - 1, 0))
    a = te_s[last]; b = tx_s[last]
    dur = torch.where(b >= 0, (b - a).clamp(min=1), torch.full_like(a, 2 * period_ns))
    cap = torch.where(b >= 0, torch.full_like(a, steps), torch.full_like(a, steps // 2))
    prog_s = torch.minimum(cap, ((tick - a).clamp(min=0) * steps) // dur)
    prog_r = torch.minimum(cap, ((tick - a).clamp(min=0) * steps + dur - 1) // dur)
    has = j > 0
    send = torch.where(has, (j - 1) * steps + prog_s, torch.zeros_like(j))
    recv = torch.where(has, (j - 1) * steps + prog_r, torch.zeros_like(j))
    return {"tick_off": torch.arange(n_ranks + 1, device=dev, dtype=torch.int64) * T, "tick_ns": tick.reshape(-1).contiguous(),
            "send_count": send.reshape(-1).to(torch.int32).contiguous(), "recv_count": recv.reshape(-1).to(torch.int32).contiguous()}
