"""Seeded synthetic rank-level communication traces.

This module only *makes inputs*: SoA columns of trace records (rank, communicator, op sequence,
op type, bytes, enter/exit timestamps, observed Send/Recv count changes) and per-rank progress
frames, shaped like what the rank probes of a 3D-parallel training job would push to the
analyzer. It holds none of the analysis arithmetic and is imported by the tests and the
benchmark, never by the oracle or by the CUDA library.

Every value is an integer computed with wrapping 64-bit integer arithmetic on torch tensors
(a counter-based hash plus fixed-point quantile tables read from `quantile_tables.json`), so
the same (spec, window) gives the same bits on the CPU and on a GPU.
"""
from .core import (  # noqa: F401
    OP_ALLREDUCE, OP_ALLGATHER, OP_REDUCESCATTER, OP_ALLTOALL, OP_SENDRECV, OP_BROADCAST,
    Family, Fault, Hang, Spec, Window, gen_window, registry, records_per_window,
)
from .ticks import gen_ticks  # noqa: F401
from .presets import cfg1, cfg2, cfg3, cfg4, cfg4w, cfg5, PRESETS  # noqa: F401
