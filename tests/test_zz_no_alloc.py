"""ccld_ring_locate_static against ccld_locate_hang and against the CPU oracle.

The static entry point serves callers that cannot allocate device memory when they need a hang
diagnosis (a watchdog thread on an out-of-memory or wedged job, a plugin inside someone else's
process). Its working memory is a fixed array inside the library that every call reuses, so the
tests make calls in a row with different answers: a result that leaked from one call's leftovers
would show up in the next. Integer results must be identical to the context-based entry point and to
the oracle's decision tree, and after the first (set-up) call on the device the amount of free device
memory must not move.
This file sorts last so that a first-failure stop has already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle as orc
import tracegen as tg
from helpers import frames_from, make_cols

pytestmark = pytest.mark.gpu

KEYS = ("cls", "n_roots_total", "n_not_entered", "n_hung", "n_not_hung", "n_missing_frames", "stuck_step", "n_members", "min_total")
ORC_KEYS = {"n_roots_total": "n_roots"}


def ring_inputs(ranks, cols, frames, n_channels, comm, seq):
    """Per ring position: rank id, state bits and progress counters, derived from an uploaded window."""
    ranks = np.asarray(ranks)
    n = len(ranks)
    c = {k: (v.cpu().numpy() if torch.is_tensor(v) else np.asarray(v)) for k, v in cols.items()}
    pos = {int(r): p for p, r in enumerate(ranks)}
    state = np.zeros(n, np.uint8)
    for i in np.nonzero((c["comm"] == comm) & (c["seq"] >= seq))[0]:
        p = pos[int(c["rank"][i])]
        state[p] |= 1
        if c["seq"][i] == seq and c["t_exit"][i] != -1:
            state[p] |= 2
    C = n_channels
    prog = np.zeros((n, max(C, 1), 2), np.int32)
    if frames is not None:
        f = {k: (v.cpu().numpy() if torch.is_tensor(v) else np.asarray(v)) for k, v in frames.items()}
        for j in np.nonzero((f["f_comm"] == comm) & (f["f_seq"] == seq))[0]:
            p = pos[int(f["f_rank"][j])]
            if not state[p] & 4:
                state[p] |= 4
                prog[p] = f["progress"][j].view(np.int32) if f["progress"].dtype != np.int32 else f["progress"][j]
    dev = torch.device("cuda", 0)
    return (torch.from_numpy(ranks.astype(np.int32)).to(dev).contiguous(), torch.from_numpy(state).to(dev),
            torch.from_numpy(prog).to(dev).contiguous() if C else None)


def check(got, want, what, orc_side=False):
    for k in KEYS:
        assert got[k] == want[ORC_KEYS.get(k, k) if orc_side else k], (what, k, got[k], want)
    assert np.array_equal(got["roots"], want["roots"]), what


def test_static_entry_point_matches_context_entry_point_twice_in_a_row():
    import paper_2605_04478_b200 as ccld
    spec = tg.cfg3(n_rings=4, ring=300, n_done=6, hung_ring=2, stuck_pos=77, n_channels=4)
    an, o = ccld.Analyzer(), orc.Oracle()
    for cid, ranks, seq0 in tg.registry(spec):
        an.comm_register(cid, ranks, 0, seq0)
        o.comm_register(cid, ranks, seq0)
    win = tg.gen_window(spec, 0, device="cuda")
    an.trace_upload(0, win.cols, win.frames, win.n_channels)
    o.upload(0, win.cols, win.frames, win.n_channels)
    an.analyze_window(0, 1, win.now_ns)
    fam = spec.families[0]
    # first the all-hung ring (H3, one root), then a ring that finished the op (H2, 300 roots), then an op
    # nobody entered (H1), then H3 again: each call must be unaffected by what the one before left behind
    for comm, seq in ((2, 6), (1, 6), (2, 7), (2, 6)):
        want = an.locate_hang(0, comm, seq)
        ranks, state, prog = ring_inputs(fam.members[comm - fam.comm_id0].numpy(), win.cols, win.frames, win.n_channels, comm, seq)
        got = ccld.ring_locate_static(ranks, state, prog)
        check(got, want, (comm, seq))
        check(got, o.locate_hang(0, comm, seq), (comm, seq, "oracle"), orc_side=True)
    assert want["cls"] == 3 and list(want["roots"]) == spec.truth["hang_root"]


def built_ring(n, kind, rng, n_channels):
    """Records and frames of one ring whose op 2 hangs, with the irregularities the decision tree must handle."""
    ranks = rng.permutation(4 * n)[:n].astype(np.int64) + 3          # ring order differs from rank order
    recs = []
    for s in range(2):
        recs += [dict(rank=int(r), comm=9, seq=s, t_enter=1000 + s, t_exit=2000 + s) for r in ranks]
    skipped = set(rng.choice(n, size=max(1, n // 7), replace=False).tolist()) if kind == "h1" else set()
    done = set(rng.choice(n, size=max(1, n // 5), replace=False).tolist()) if kind == "h2" else set()
    for p, r in enumerate(ranks):
        if p in skipped:
            if p % 2 == 0 and p != min(skipped):                       # some of them are already past the op
                recs.append(dict(rank=int(r), comm=9, seq=3, t_enter=5000, t_exit=-1))
            continue
        recs.append(dict(rank=int(r), comm=9, seq=2, t_enter=4000, t_exit=(4100 if p in done else -1)))
    entries = []
    if n_channels:
        base = int(rng.integers(5, 50))
        tot = np.full(n, base + 1)
        if kind == "h3_tied":                                          # a run of equal minima that wraps around the ring
            for p in (n - 2, n - 1, 0, 1):
                tot[p % n] = base
        elif kind == "h3_equal":
            tot[:] = base
        else:
            tot[int(rng.integers(0, n))] = base
        missing = set(rng.choice(n, size=n // 9, replace=False).tolist()) if kind == "h3_missing" else set()
        for p, r in enumerate(ranks):
            if p not in missing:
                entries.append((int(r), 9, 2, [(int(tot[p]), int(tot[p]) - (ch % 2)) for ch in range(n_channels)]))
        entries.append((int(ranks[0]), 9, 1, [(1, 1)] * n_channels))     # a frame of another op is ignored
    return ranks, recs, (frames_from(entries, n_channels) if n_channels else None)


@pytest.mark.parametrize("n", [1, 2, 300, 1025, 3000, 8192])
def test_static_entry_point_on_built_rings_of_every_size(n):
    """H1 with members already past the op, H2, H3 with a unique minimum, a wrapping run of minima, all equal, members
    without a frame, and no progress table at all; rings below, at and far above the CTA size; a root list shorter than
    the answer. Static entry point = context entry point = oracle, call after call on the same scratch array."""
    import paper_2605_04478_b200 as ccld
    rng = np.random.default_rng(n)
    for kind, C in (("h3", 3), ("h1", 2), ("h3_tied", 1), ("h2", 2), ("h3_missing", 4), ("h3_equal", 2), ("h3", 0), ("h1", 0)):
        ranks, recs, frames = built_ring(n, kind, rng, C)
        cols = make_cols(recs)
        an, o = ccld.Analyzer(), orc.Oracle()
        an.comm_register(9, ranks, 0, 0)
        o.comm_register(9, ranks, 0)
        an.trace_upload(0, cols, frames, C)
        o.upload(0, cols, frames, C)
        an.analyze_window(0, 1, 10**6)
        want, ow = an.locate_hang(0, 9, 2), o.locate_hang(0, 9, 2)
        d_ranks, d_state, d_prog = ring_inputs(ranks, cols, frames, C, 9, 2)
        got = ccld.ring_locate_static(d_ranks, d_state, d_prog)
        check(got, want, (n, kind, C))
        check(got, ow, (n, kind, C, "oracle"), orc_side=True)
        assert got["cls"] == {"h1": 1, "h2": 2}.get(kind, 3)
        # a root list that is too short is filled as far as it goes and the total still says how many there are
        short = ccld.ring_locate_static(d_ranks, d_state, d_prog, roots_cap=1)
        assert short["n_roots_total"] == want["n_roots_total"] and list(short["roots"]) == list(want["roots"][:1])
        an.close()


def test_static_entry_point_leaves_free_device_memory_unchanged():
    """After the set-up call on the device, calls must not take or return device memory: the free byte count that the
    driver reports stays where it was across many calls of changing size."""
    import paper_2605_04478_b200 as ccld
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(3)
    cases = []
    for n in (1, 77, 1024, 1025, 8192):
        ranks = torch.arange(n, dtype=torch.int32, device=dev)
        state = torch.from_numpy((rng.integers(0, 2, n) * 2 + 5).astype(np.uint8)).to(dev)      # entered, framed, some complete
        prog = torch.from_numpy(rng.integers(0, 90, (n, 2, 2)).astype(np.int32)).to(dev)
        cases.append((ranks, state, prog))
    ccld.ring_locate_static(*cases[0])                                # set-up call: context, module, symbol address
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(20):
        for c in cases:
            ccld.ring_locate_static(*c)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, (free0, free1)


def test_static_entry_point_rejects_oversized_rings():
    import paper_2605_04478_b200 as ccld
    n = ccld.STATIC_MAX_MEMBERS + 1
    dev = torch.device("cuda", 0)
    with pytest.raises(ccld.CcldError) as e:
        ccld.ring_locate_static(torch.arange(n, dtype=torch.int32, device=dev), torch.zeros(n, dtype=torch.uint8, device=dev))
    assert e.value.code == -8 and "CCLD_STATIC_MAX_MEMBERS" in str(e.value)
