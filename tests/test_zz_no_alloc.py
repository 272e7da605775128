"""ccld_ring_locate_static against ccld_locate_hang.

The static entry point serves callers that cannot allocate device memory when they need a hang
diagnosis (a watchdog on an out-of-memory or wedged job, a plugin inside someone else's process).
Its working memory is a fixed array inside the library that every call reuses, so the test makes
two calls in a row with different answers: a result that leaked from the first call's leftovers
would show up in the second. Integer results must be identical to the context-based entry point.
This file sorts last so that a first-failure stop has already run every other test.
"""
import numpy as np
import pytest
import torch

import tracegen as tg

pytestmark = pytest.mark.gpu

KEYS = ("cls", "n_roots_total", "n_not_entered", "n_hung", "n_not_hung", "n_missing_frames", "stuck_step", "n_members", "min_total")


def ring_inputs(spec, win, comm, seq):
    """Per ring position: rank id, state bits and progress counters, derived from the uploaded window."""
    fam = spec.families[0]
    ranks = fam.members[comm - fam.comm_id0]
    n = len(ranks)
    c = {k: v.cpu().numpy() for k, v in win.cols.items()}
    pos = {int(r): p for p, r in enumerate(ranks)}
    state = np.zeros(n, np.uint8)
    for i in np.nonzero((c["comm"] == comm) & (c["seq"] >= seq))[0]:
        p = pos[int(c["rank"][i])]
        state[p] |= 1
        if c["seq"][i] == seq and c["t_exit"][i] != -1:
            state[p] |= 2
    C = win.n_channels
    prog = np.zeros((n, max(C, 1), 2), np.int32)
    if win.frames is not None:
        f = {k: v.cpu().numpy() for k, v in win.frames.items()}
        for j in np.nonzero((f["f_comm"] == comm) & (f["f_seq"] == seq))[0]:
            p = pos[int(f["f_rank"][j])]
            if not state[p] & 4:
                state[p] |= 4
                prog[p] = f["progress"][j]
    dev = torch.device("cuda", 0)
    return (ranks.to(torch.int32).to(dev).contiguous(), torch.from_numpy(state).to(dev),
            torch.from_numpy(prog).to(dev).contiguous() if C else None)


def test_static_entry_point_matches_context_entry_point_twice_in_a_row():
    import paper_2605_04478_b200 as ccld
    spec = tg.cfg3(n_rings=4, ring=300, n_done=6, hung_ring=2, stuck_pos=77, n_channels=4)
    an = ccld.Analyzer()
    for cid, ranks, seq0 in tg.registry(spec):
        an.comm_register(cid, ranks, 0, seq0)
    win = tg.gen_window(spec, 0, device="cuda")
    an.trace_upload(0, win.cols, win.frames, win.n_channels)
    an.analyze_window(0, 1, win.now_ns)
    # first the all-hung ring (H3, one root), then a ring that finished the op (H2, 300 roots), then an op
    # nobody entered (H1), then H3 again: each call must be unaffected by what the one before left behind
    for comm, seq in ((2, 6), (1, 6), (2, 7), (2, 6)):
        want = an.locate_hang(0, comm, seq)
        ranks, state, prog = ring_inputs(spec, win, comm, seq)
        got = ccld.ring_locate_static(ranks, state, prog)
        for k in KEYS:
            assert got[k] == want[k], (comm, seq, k, got[k], want[k])
        assert np.array_equal(got["roots"], want["roots"]), (comm, seq)
    assert want["cls"] == 3 and list(want["roots"]) == spec.truth["hang_root"]


def test_static_entry_point_rejects_oversized_rings():
    import paper_2605_04478_b200 as ccld
    n = ccld.STATIC_MAX_MEMBERS + 1
    dev = torch.device("cuda", 0)
    with pytest.raises(ccld.CcldError) as e:
        ccld.ring_locate_static(torch.arange(n, dtype=torch.int32, device=dev), torch.zeros(n, dtype=torch.uint8, device=dev))
    assert e.value.code == -8 and "CCLD_STATIC_MAX_MEMBERS" in str(e.value)
