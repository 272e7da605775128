"""Python binding of libccld, the B200 (sm_100a) implementation of the CCL-D decision-analyzer hot path.

Argument marshalling only: every step of the analysis runs in the CUDA kernels of the C-ABI library
`libccld.so` (declared in include/ccld.h). PyTorch supplies device memory and the CUDA stream.
There is no CPU path: importing works anywhere, but creating an Analyzer needs the built library
and a CUDA device and raises otherwise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libccld.so")

OK = 0
ERRORS = {-1: "ARG", -2: "NOMEM", -3: "CUDA", -4: "UNKNOWN_COMM", -5: "NOT_MEMBER", -6: "SEQ_RANGE",
          -7: "NO_WINDOW", -8: "CAPACITY", -9: "STATE", -10: "DUPLICATE"}
MAX_COMM_SIZE = 8192
MAX_ALERTS_PER_WINDOW = 1024

EXPORTS = ("ccld_params_default", "ccld_create", "ccld_destroy", "ccld_last_error", "ccld_comm_register",
           "ccld_trace_upload", "ccld_window_release", "ccld_analyze_window", "ccld_reset", "ccld_get_verdict",
           "ccld_locate_hang", "ccld_get_optable", "ccld_get_ranges", "ccld_get_rank_stats", "ccld_copy_to_host",
           "ccld_timing_enable", "ccld_get_kernel_times", "ccld_set_speculation", "ccld_ring_locate_static", "ccld_derive_rates", "ccld_locate_hangs", "ccld_state_export", "ccld_state_import", "ccld_trace_attach_opset", "ccld_opset_check",
           "ccld_comm_set_layers")
STATIC_MAX_MEMBERS = 8192
KERNEL_KINDS = ("k_seq_range", "k_plan", "k_slot_scatter", "k_reduce_fused", "k_reduce_mid", "k_reduce_large", "k_window_decide")


class CcldError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"ccld error {code} ({ERRORS.get(code, '?')}): {msg}")
        self.code = code


class Params(C.Structure):
    _fields_ = [("tbase_init_ns", C.c_int64), ("theta_slow_milli", C.c_uint32), ("alpha_milli", C.c_uint32),
                ("beta_milli", C.c_uint32), ("m_max_rounds", C.c_uint32), ("m_max_ns", C.c_int64),
                ("hang_ns", C.c_int64), ("barrier_bytes", C.c_uint64), ("slow_rep_threshold", C.c_uint32),
                ("k_milli", C.c_uint32), ("min_group", C.c_uint32), ("vote_rep_milli", C.c_uint32)]


class Suspect(C.Structure):
    _fields_ = [("kind", C.c_uint32), ("rank", C.c_uint32), ("votes", C.c_uint32), ("ops", C.c_uint32),
                ("mean_busbw", C.c_double)]


class CommVerdict(C.Structure):
    _fields_ = [(k, C.c_uint32) for k in ("comm", "n_rounds", "sel_seq", "cls", "slow_detected", "located",
                                           "baseline_static", "rate_source", "root_comp", "root_comm")] + \
               [(k, C.c_uint64) for k in ("slow_count", "rounds_total", "m")] + \
               [(k, C.c_int64) for k in ("t_max", "t_min", "t_base")] + [("R", C.c_double), ("P", C.c_double)]


class HangAlert(C.Structure):
    _fields_ = [("comm", C.c_uint32), ("seq", C.c_uint32), ("age_ns", C.c_int64)]


class Verdict(C.Structure):
    _fields_ = [(k, C.c_uint64) for k in ("n_records", "n_groups", "n_slots", "n_rejected", "n_complete", "n_incomplete",
                                           "n_barrier", "n_analysed", "n_flag_skew", "n_flag_dur", "n_opset_mismatch")] + \
               [(k, C.c_uint32) for k in ("error_bits", "n_comm_rows_total", "n_alerts_total", "n_suspects_total")] + \
               [("comm_rows", C.POINTER(CommVerdict)), ("comm_rows_cap", C.c_uint32),
                ("alerts", C.POINTER(HangAlert)), ("alerts_cap", C.c_uint32),
                ("suspects", C.POINTER(Suspect)), ("suspects_cap", C.c_uint32)]


class HangVerdict(C.Structure):
    _fields_ = [(k, C.c_uint32) for k in ("cls", "n_roots_total", "n_not_entered", "n_hung", "n_not_hung",
                                           "n_missing_frames", "stuck_step", "n_members")] + \
               [("min_total", C.c_uint64), ("roots", C.POINTER(C.c_uint32)), ("roots_cap", C.c_uint32)]


OPTABLE_I64 = ("e_min", "arrival_skew", "t_max", "t_min", "span", "med_skew", "mad_skew", "med_dur", "mad_dur")
OPTABLE_U32 = ("rank_tmin", "rank_tmax", "max_chg", "rank_max_chg", "n_present", "gflags")


class OpsetVerdict(C.Structure):
    _fields_ = [(k, C.c_uint32) for k in ("n_members", "n_present", "n_deviating_total", "majority_count")] + \
               [(k, C.c_uint8) for k in ("op", "algo", "proto", "pad")] + \
               [("bytes", C.c_uint64), ("ranks", C.POINTER(C.c_uint32)), ("ranks_cap", C.c_uint32)]


class OpTable(C.Structure):
    _fields_ = [("n_groups", C.c_uint64), ("n_slots", C.c_uint64)] + [(k, C.c_void_p) for k in OPTABLE_I64] + \
               [(k, C.c_void_p) for k in OPTABLE_U32] + [("busbw", C.c_void_p), ("flags", C.c_void_p), ("perm", C.c_void_p)]


class CommRange(C.Structure):
    _fields_ = [("comm", C.c_uint32), ("n", C.c_uint32), ("seq_lo", C.c_uint32), ("n_seq", C.c_uint32),
                ("group0", C.c_uint64), ("slot0", C.c_uint64)]


_NP_OF = {C.c_uint32: "u4", C.c_uint64: "u8", C.c_int64: "i8", C.c_double: "f8"}
_lib = None


def load_library() -> C.CDLL:
    """Loads libccld.so; raises if it has not been built (python -m paper_2605_04478_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2605_04478_b200.build`; "
                               "there is no fallback path")
        lib = C.CDLL(LIB_PATH)
        for name in EXPORTS:
            getattr(lib, name).restype = C.c_int
        lib.ccld_params_default.restype = None
        lib.ccld_params_default.argtypes = [C.POINTER(Params)]
        lib.ccld_last_error.restype = C.c_char_p
        lib.ccld_last_error.argtypes = [C.c_void_p]
        lib.ccld_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(Params), C.c_int, C.c_void_p]
        lib.ccld_destroy.argtypes = [C.c_void_p]
        lib.ccld_comm_register.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32, C.c_uint8, C.c_uint32]
        lib.ccld_comm_set_layers.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p]
        lib.ccld_trace_upload.argtypes = [C.c_void_p, C.c_uint32, C.c_uint64, C.c_int] + [C.c_void_p] * 9 + \
                                         [C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p]
        lib.ccld_window_release.argtypes = [C.c_void_p, C.c_uint32]
        lib.ccld_analyze_window.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.c_int64]
        lib.ccld_reset.argtypes = [C.c_void_p]
        lib.ccld_set_speculation.argtypes = [C.c_void_p, C.c_int]
        lib.ccld_get_verdict.argtypes = [C.c_void_p, C.c_uint32, C.POINTER(Verdict)]
        lib.ccld_locate_hang.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint32, C.POINTER(HangVerdict)]
        lib.ccld_trace_attach_opset.argtypes = [C.c_void_p, C.c_uint32, C.c_int, C.c_void_p, C.c_void_p]
        lib.ccld_opset_check.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint32, C.POINTER(OpsetVerdict)]
        lib.ccld_state_export.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.POINTER(C.c_uint64)]
        lib.ccld_state_import.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64]
        lib.ccld_locate_hangs.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32, C.POINTER(C.c_uint32)]
        lib.ccld_get_optable.argtypes = [C.c_void_p, C.c_uint32, C.POINTER(OpTable)]
        lib.ccld_get_ranges.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32, C.POINTER(C.c_uint32)]
        lib.ccld_get_rank_stats.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.ccld_copy_to_host.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64]
        lib.ccld_derive_rates.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint64] + [C.c_void_p] * 6
        lib.ccld_timing_enable.argtypes = [C.c_void_p, C.c_int]
        lib.ccld_get_kernel_times.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        lib.ccld_ring_locate_static.argtypes = [C.c_int, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p,
                                                C.POINTER(HangVerdict), C.c_char_p, C.c_uint32]
        _lib = lib
    return _lib


def default_params() -> Params:
    p = Params()
    load_library().ccld_params_default(C.byref(p))
    return p


_COL_DTYPES = {"rank": "int32", "comm": "int32", "seq": "int32", "op": "uint8", "bytes": "int64",
               "t_enter": "int64", "t_exit": "int64", "send_chg": "int32", "recv_chg": "int32"}


def _as_tensor(torch, v, dt):
    """numpy / list -> torch tensor of dtype dt (same bits for unsigned inputs of equal width)."""
    if torch.is_tensor(v):
        return v
    a = np.ascontiguousarray(v)
    if a.dtype != np.dtype(dt):
        a = a.view(dt) if a.dtype.itemsize == np.dtype(dt).itemsize else a.astype(dt)
    return torch.from_numpy(a)


def ring_locate_static(ranks, state, progress=None, device: int = 0, stream=None, roots_cap: int = STATIC_MAX_MEMBERS):
    """Hang location for one ring through ccld_ring_locate_static, the entry point that allocates nothing.

    For callers that cannot allocate device memory at diagnosis time (out-of-memory or wedged-allocator
    watchdogs, plugins hosted in another process, tight monitoring loops). ranks (int32 [n]), state
    (uint8 [n]: bit0 entered, bit1 complete, bit2 has a frame) and progress (int32 [n, channels, 2] or
    None) are CUDA tensors the caller already owns, in ring order. This wrapper itself only builds small
    host-side ctypes objects. Calls on one device share a fixed scratch array: do not overlap them.
    """
    lib = load_library()
    n = int(ranks.numel())
    assert ranks.is_cuda and state.is_cuda and ranks.is_contiguous() and state.is_contiguous()
    n_ch = 0 if progress is None else int(progress.shape[1])
    roots = (C.c_uint32 * max(roots_cap, 1))()
    hv = HangVerdict()
    hv.roots = C.cast(roots, C.POINTER(C.c_uint32)); hv.roots_cap = roots_cap
    err = C.create_string_buffer(256)
    rc = lib.ccld_ring_locate_static(device, C.c_void_p(stream.cuda_stream if stream is not None else 0), n,
                                     C.c_void_p(ranks.data_ptr()), C.c_void_p(state.data_ptr()), n_ch,
                                     C.c_void_p(progress.data_ptr() if progress is not None else 0), C.byref(hv), err, 256)
    if rc != OK:
        raise CcldError(rc, err.value.decode())
    out: Dict[str, object] = {k: int(getattr(hv, k)) for k in ("cls", "n_roots_total", "n_not_entered", "n_hung", "n_not_hung",
                                                             "n_missing_frames", "stuck_step", "n_members", "min_total")}
    out["roots"] = np.array(roots[:min(hv.n_roots_total, roots_cap)], dtype=np.uint32)
    return out


class Analyzer:
    """One analysis context on one GPU. Method names follow the C entry points."""

    def __init__(self, params: Optional[Dict[str, int]] = None, device: int = 0, stream=None):
        import torch
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the analyzer has no CPU path")
        self.torch = torch
        self.device = device
        p = default_params()
        for k, v in (params or {}).items():
            if not hasattr(p, k):
                raise KeyError(k)
            setattr(p, k, v)
        self.params = p
        self._stream = stream
        sh = C.c_void_p(stream.cuda_stream if stream is not None else 0)
        self.h = C.c_void_p()
        rc = self.lib.ccld_create(C.byref(self.h), C.byref(p), device, sh)
        if rc != OK:
            raise CcldError(rc, "ccld_create failed")
        self._keep: Dict[int, list] = {}

    # -- helpers
    def _check(self, rc: int):
        if rc != OK:
            raise CcldError(rc, self.lib.ccld_last_error(self.h).decode())

    def close(self):
        if getattr(self, "h", None) is not None and self.h.value:
            self.lib.ccld_destroy(self.h)
            self.h = C.c_void_p()
            self._keep.clear()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _to_host(self, ptr, count: int, dtype) -> np.ndarray:
        out = np.empty(count, dtype=dtype)
        if count:
            self._check(self.lib.ccld_copy_to_host(self.h, out.ctypes.data, ptr, out.nbytes))
        return out

    # -- the boundary
    def comm_register(self, comm: int, ranks, algo: int = 0, seq0: int = 0) -> None:
        r = np.ascontiguousarray(np.asarray(ranks, dtype=np.uint32))
        self._check(self.lib.ccld_comm_register(self.h, comm, r.ctypes.data, len(r), algo, seq0))

    def comm_set_layers(self, comm: int, layers) -> None:
        a = np.ascontiguousarray(np.asarray(layers, dtype=np.uint32))
        self._check(self.lib.ccld_comm_set_layers(self.h, comm, a.ctypes.data))

    def trace_upload(self, window_id: int, cols, frames=None, n_channels: int = 0) -> None:
        """cols: dict of torch tensors or numpy arrays, all on the CPU (copied) or all on this GPU (borrowed)."""
        torch = self.torch
        t = {}
        for k, dt in _COL_DTYPES.items():
            v = cols.get(k)
            if v is None:
                t[k] = None
                continue
            v = _as_tensor(torch, v, dt)
            assert str(v.dtype) == "torch." + dt, (k, v.dtype)
            t[k] = v.contiguous()
        devs = {v.device.type for v in t.values() if v is not None}
        fr = {}
        if frames is not None:
            for k in ("f_rank", "f_comm", "f_seq", "progress"):
                fr[k] = _as_tensor(torch, frames[k], "int32").contiguous()
                devs.add(fr[k].device.type)
        assert len(devs) == 1, "all columns must live on the same device"
        mem_kind = 1 if devs.pop() == "cuda" else 0
        n = int(t["rank"].numel())
        ptr = lambda v: C.c_void_p(v.data_ptr()) if v is not None and v.numel() else C.c_void_p(0)
        nf = int(fr["f_rank"].numel()) if fr else 0
        rc = self.lib.ccld_trace_upload(self.h, window_id, n, mem_kind, ptr(t["rank"]), ptr(t["comm"]), ptr(t["seq"]), ptr(t["op"]),
                                        ptr(t["bytes"]), ptr(t["t_enter"]), ptr(t["t_exit"]), ptr(t["send_chg"]), ptr(t["recv_chg"]),
                                        nf, ptr(fr.get("f_rank")), ptr(fr.get("f_comm")), ptr(fr.get("f_seq")), n_channels,
                                        ptr(fr.get("progress")))
        self._check(rc)
        self._keep[window_id] = [t, fr]            # borrowed device memory / pinned host memory stays alive

    def window_release(self, window_id: int) -> None:
        self._check(self.lib.ccld_window_release(self.h, window_id))
        self._keep.pop(window_id, None)
        self._keep.pop(("opset", window_id), None)

    def analyze_window(self, first_window: int, n_windows: int, now_ns: int) -> None:
        self._check(self.lib.ccld_analyze_window(self.h, first_window, n_windows, now_ns))

    def reset(self) -> None:
        self._check(self.lib.ccld_reset(self.h))

    def set_speculation(self, on: bool) -> None:
        self._check(self.lib.ccld_set_speculation(self.h, 1 if on else 0))

    @staticmethod
    def _records(buf, struct, count, cap):
        dt = np.dtype([(k, _NP_OF[t]) for k, t in struct._fields_])
        a = np.frombuffer(buf, dtype=dt, count=max(cap, 1))[:count]
        return {k: a[k].copy() for k in dt.names}

    def get_verdict(self, window_id: int, comm_rows_cap: int = 1 << 16, alerts_cap: int = MAX_ALERTS_PER_WINDOW,
                    suspects_cap: int = 1 << 16, check: bool = True) -> Dict[str, object]:
        rows = (CommVerdict * max(comm_rows_cap, 1))()
        alerts = (HangAlert * max(alerts_cap, 1))()
        sus = (Suspect * max(suspects_cap, 1))()
        v = Verdict()
        v.comm_rows = C.cast(rows, C.POINTER(CommVerdict)); v.comm_rows_cap = comm_rows_cap
        v.alerts = C.cast(alerts, C.POINTER(HangAlert)); v.alerts_cap = alerts_cap
        v.suspects = C.cast(sus, C.POINTER(Suspect)); v.suspects_cap = suspects_cap
        rc = self.lib.ccld_get_verdict(self.h, window_id, C.byref(v))
        if check:
            self._check(rc)
        out: Dict[str, object] = {k: int(getattr(v, k)) for k, _ in Verdict._fields_[:15]}
        out["rc"] = rc
        out["comm_rows"] = self._records(rows, CommVerdict, min(v.n_comm_rows_total, comm_rows_cap), comm_rows_cap)
        out["alerts"] = self._records(alerts, HangAlert, min(v.n_alerts_total, alerts_cap, MAX_ALERTS_PER_WINDOW), alerts_cap)
        out["suspects"] = self._records(sus, Suspect, min(v.n_suspects_total, suspects_cap), suspects_cap)
        return out

    def locate_hang(self, window_id: int, comm: int, seq: int, roots_cap: int = MAX_COMM_SIZE) -> Dict[str, object]:
        roots = (C.c_uint32 * max(roots_cap, 1))()
        hv = HangVerdict()
        hv.roots = C.cast(roots, C.POINTER(C.c_uint32)); hv.roots_cap = roots_cap
        self._check(self.lib.ccld_locate_hang(self.h, window_id, comm, seq, C.byref(hv)))
        out: Dict[str, object] = {k: int(getattr(hv, k)) for k in ("cls", "n_roots_total", "n_not_entered", "n_hung", "n_not_hung",
                                                                 "n_missing_frames", "stuck_step", "n_members", "min_total")}
        out["roots"] = np.array(roots[:min(hv.n_roots_total, roots_cap)], dtype=np.uint32)
        return out

    def locate_hangs(self, window_id: int, cap: int = 1024, roots_stride: int = 64) -> List[Dict[str, object]]:
        """ccld_locate_hangs: the hang verdict of every alert of the window, one launch; each dict also carries the alert's
        comm, seq and age_ns."""
        n = C.c_uint32(0)
        cap = max(cap, 1)
        hv = (HangVerdict * cap)(); al = (HangAlert * cap)()
        roots = (C.c_uint32 * (cap * max(roots_stride, 1)))()
        self._check(self.lib.ccld_locate_hangs(self.h, window_id, C.cast(al, C.c_void_p), C.cast(hv, C.c_void_p), cap,
                                               C.cast(roots, C.c_void_p), roots_stride, C.byref(n)))
        res = []
        for i in range(min(n.value, cap)):
            d: Dict[str, object] = {k: int(getattr(hv[i], k)) for k in ("cls", "n_roots_total", "n_not_entered", "n_hung", "n_not_hung",
                                                                      "n_missing_frames", "stuck_step", "n_members", "min_total")}
            k = min(hv[i].n_roots_total, roots_stride)
            d["roots"] = np.array(roots[i * roots_stride:i * roots_stride + k], dtype=np.uint32)
            d["comm"], d["seq"], d["age_ns"] = int(al[i].comm), int(al[i].seq), int(al[i].age_ns)
            res.append(d)
        return res

    def trace_attach_opset(self, window_id: int, algo, proto) -> None:
        """ccld_trace_attach_opset: algorithm and protocol codes per record (uint8), host (copied) or this GPU (borrowed)."""
        torch = self.torch
        a = _as_tensor(torch, algo, "uint8").contiguous(); b = _as_tensor(torch, proto, "uint8").contiguous()
        assert a.device.type == b.device.type
        self._check(self.lib.ccld_trace_attach_opset(self.h, window_id, 1 if a.device.type == "cuda" else 0,
                                                     C.c_void_p(a.data_ptr()), C.c_void_p(b.data_ptr())))
        self._keep.setdefault(("opset", window_id), []).append((a, b))

    def opset_check(self, window_id: int, comm: int, seq: int, ranks_cap: int = MAX_COMM_SIZE) -> Dict[str, object]:
        """ccld_opset_check: majority Operation Type Set of op (comm, seq) and the ranks that deviate from it."""
        ranks = (C.c_uint32 * max(ranks_cap, 1))()
        v = OpsetVerdict()
        v.ranks = C.cast(ranks, C.POINTER(C.c_uint32)); v.ranks_cap = ranks_cap
        self._check(self.lib.ccld_opset_check(self.h, window_id, comm, seq, C.byref(v)))
        out: Dict[str, object] = {k: int(getattr(v, k)) for k in ("n_members", "n_present", "n_deviating_total", "majority_count",
                                                                "op", "algo", "proto", "bytes")}
        out["ranks"] = np.array(ranks[:min(v.n_deviating_total, ranks_cap)], dtype=np.uint32)
        return out

    def state_export(self) -> bytes:
        """ccld_state_export: the cumulative state (Eq. 1 baselines, repetition counters, per-rank votes and sums) as bytes."""
        n = C.c_uint64(0)
        self._check(self.lib.ccld_state_export(self.h, None, 0, C.byref(n)))
        buf = (C.c_char * n.value)()
        self._check(self.lib.ccld_state_export(self.h, C.cast(buf, C.c_void_p), n.value, C.byref(n)))
        return bytes(buf)

    def state_import(self, blob: bytes) -> None:
        buf = (C.c_char * len(blob)).from_buffer_copy(blob)
        self._check(self.lib.ccld_state_import(self.h, C.cast(buf, C.c_void_p), len(blob)))

    def get_ranges(self, window_id: int) -> Dict[str, np.ndarray]:
        n = C.c_uint32(0)
        self._check(self.lib.ccld_get_ranges(self.h, window_id, None, 0, C.byref(n)))
        rows = (CommRange * max(n.value, 1))()
        self._check(self.lib.ccld_get_ranges(self.h, window_id, C.cast(rows, C.c_void_p), n.value, C.byref(n)))
        return self._records(rows, CommRange, n.value, n.value)

    def get_optable(self, window_id: int, to_host: bool = True) -> Dict[str, object]:
        """Per-op table of an analysed window; with to_host the columns come back as numpy arrays."""
        t = OpTable()
        self._check(self.lib.ccld_get_optable(self.h, window_id, C.byref(t)))
        G, S = int(t.n_groups), int(t.n_slots)
        if not to_host:
            return {k: getattr(t, k) for k, _ in OpTable._fields_}
        out: Dict[str, object] = {"n_groups": G, "n_slots": S}
        for k in OPTABLE_I64:
            out[k] = self._to_host(getattr(t, k), G, np.int64)
        for k in OPTABLE_U32:
            out[k] = self._to_host(getattr(t, k), G, np.uint32)
        out["busbw"] = self._to_host(t.busbw, G, np.float64)
        out["flags"] = self._to_host(t.flags, S, np.uint8)
        out["perm"] = self._to_host(t.perm, S, np.uint32)
        # per-group communicator id, op counter and first slot, expanded from the range rows
        r = self.get_ranges(window_id)
        ns = r["n_seq"].astype(np.int64)
        within = np.arange(int(ns.sum()), dtype=np.int64) - np.repeat(np.cumsum(ns) - ns, ns)
        out["comm"] = np.repeat(r["comm"], ns).astype(np.uint32)
        out["seq"] = (np.repeat(r["seq_lo"].astype(np.int64), ns) + within).astype(np.uint32)
        out["slot0"] = (np.repeat(r["slot0"].astype(np.int64), ns) + within * np.repeat(r["n"].astype(np.int64), ns)).astype(np.uint64)
        return out

    def timing_enable(self, on: bool = True) -> None:
        self._check(self.lib.ccld_timing_enable(self.h, 1 if on else 0))

    def get_kernel_times(self) -> Dict[str, Dict[str, float]]:
        """Per kernel kind: summed device milliseconds and launches since timing was enabled."""
        ms = np.zeros(len(KERNEL_KINDS), np.float64); n = np.zeros(len(KERNEL_KINDS), np.uint64)
        self._check(self.lib.ccld_get_kernel_times(self.h, ms.ctypes.data, n.ctypes.data))
        return {k: {"ms": float(ms[i]), "launches": int(n[i])} for i, k in enumerate(KERNEL_KINDS)}

    def derive_rates(self, rank, t_enter, t_exit, tick_off, tick_ns, send_count, recv_count):
        """ccld_derive_rates: counter changes per record from raw probe samples (Sec. 4.1.2). All inputs are tensors on
        this GPU; returns (send_chg, recv_chg) as int32 tensors on this GPU (bit pattern uint32), written asynchronously on
        the analyzer's stream."""
        torch = self.torch
        cols = [_as_tensor(torch, rank, "int32"), _as_tensor(torch, t_enter, "int64"), _as_tensor(torch, t_exit, "int64"),
                _as_tensor(torch, tick_off, "int64"), _as_tensor(torch, tick_ns, "int64"), _as_tensor(torch, send_count, "int32"),
                _as_tensor(torch, recv_count, "int32")]
        assert all(c.device.type == "cuda" for c in cols), "ccld_derive_rates takes device memory"
        cols = [c.contiguous() for c in cols]
        n = int(cols[0].numel()); n_ranks = int(cols[3].numel()) - 1; n_ticks = int(cols[4].numel())
        out_s = torch.empty(n, dtype=torch.int32, device=cols[0].device); out_r = torch.empty_like(out_s)
        ptr = lambda v: C.c_void_p(v.data_ptr()) if v.numel() else C.c_void_p(0)
        self._check(self.lib.ccld_derive_rates(self.h, n, ptr(cols[0]), ptr(cols[1]), ptr(cols[2]), n_ranks, n_ticks, ptr(cols[3]),
                                               ptr(cols[4]), ptr(cols[5]), ptr(cols[6]), ptr(out_s), ptr(out_r)))
        self._rate_keep = cols                     # inputs stay alive until the next call or a synchronization
        return out_s, out_r

    def get_rank_stats(self, n_ranks: int) -> Dict[str, np.ndarray]:
        votes = np.zeros((n_ranks, 4), np.uint32); ops = np.zeros(n_ranks, np.uint32)
        cnt = np.zeros(n_ranks, np.uint32); bw = np.zeros(n_ranks, np.float64)
        self._check(self.lib.ccld_get_rank_stats(self.h, n_ranks, votes.ctypes.data, ops.ctypes.data, cnt.ctypes.data, bw.ctypes.data))
        return {"votes": votes, "ops": ops, "bw_cnt": cnt, "bw_sum": bw}
