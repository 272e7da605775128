"""The C-ABI library loads and exports every entry point include/ccld.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    src = open(os.path.join(ROOT, "include", "ccld.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(ccld_[a-z_]+)\s*\(", src)))


def test_header_declares_the_four_named_calls():
    names = declared_functions()
    for n in ("ccld_trace_upload", "ccld_analyze_window", "ccld_locate_hang", "ccld_get_verdict"):
        assert n in names


def test_library_exports_every_declared_symbol():
    import paper_2605_04478_b200 as ccld
    from paper_2605_04478_b200.build import build
    build()
    lib = ctypes.CDLL(ccld.LIB_PATH)
    names = declared_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(ccld.EXPORTS) == names


def test_defaults_and_struct_sizes():
    import paper_2605_04478_b200 as ccld
    from paper_2605_04478_b200.build import build
    build()
    p = ccld.default_params()
    assert (p.theta_slow_milli, p.alpha_milli, p.beta_milli, p.m_max_rounds) == (3000, 400, 600, 100)
    assert p.m_max_ns == 120 * 10**9 and p.hang_ns == 300 * 10**9 and p.barrier_bytes == 4
    # sizes of the C structs on this ABI (x86-64 / aarch64 LP64)
    want = dict(CommVerdict=104, Suspect=24, HangAlert=16, CommRange=32, Params=64, Verdict=152, HangVerdict=56, OpTable=160)
    for k, v in want.items():
        assert ctypes.sizeof(getattr(ccld, k)) == v, k


def test_no_cpu_fallback():
    import torch
    import paper_2605_04478_b200 as ccld
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        ccld.Analyzer()
    # the product package never refers to the oracle
    pkg = os.path.dirname(ccld.__file__)
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                assert "oracle" not in open(os.path.join(dirpath, f)).read().lower(), f
