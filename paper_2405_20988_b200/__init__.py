"""B200-native FDA monitoring / synchronisation library: thin Python binding over libfda.

Only argument marshalling lives here; every step of the path runs in the CUDA kernels of
``libfda.so`` (built by ``python -m paper_2405_20988_b200.build``).  Importing the package
does not load the library; the first call does, and fails loudly if it is missing.
"""
from .binding import (  # noqa: F401
    FDA_AVG_BROADCAST,
    FDA_AVG_UNCONDITIONAL,
    FDA_STATE_LINEAR,
    FDA_STATE_NORM,
    FDA_STATE_SKETCH,
    FDA_VARIANT_LINEAR,
    FDA_VARIANT_SKETCH,
    Estimate,
    FdaContext,
    FdaError,
    fda_local_state_linear_noalloc,
    FDA_NOALLOC_MAX_WORKERS,
    library_path,
    load_library,
)
from .rounds import run_rounds  # noqa: F401
