"""fp64 CPU oracle for decode attention over a layer-shared KV cache.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this; only
the tests, the smoke check and the benchmark's CPU-baseline leg do.  The
arithmetic lives in ``kvs_oracle.c`` (plain C, compiled here with gcc); this
module is a ctypes wrapper that moves numpy float64 arrays in and out.
"""
from .oracle import (  # noqa: F401
    Oracle,
    attend_unit,
    attend_units,
    build,
    combine_partials,
    mean_cosine,
    num_threads,
    partial_unit,
    slot_table,
)
