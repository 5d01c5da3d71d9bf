"""CPU oracle for the FDA hot path (test infrastructure only).

Thin ctypes access to ``fda_oracle.c``: the plain fp64 statement of the local state
(drift norm, projection, AMS sketch), the averaged-state estimate H with its trigger and
the K-way model average, written from the paper's Section 3.  Nothing here is part of the
product: only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package, and it imports nothing from the CUDA library.
"""
from .fda_oracle import (  # noqa: F401
    P61,
    build,
    hash_dump,
    local_state,
    combine,
    average,
    variance,
    direction,
    state_len,
)
