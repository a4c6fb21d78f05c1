"""B200-native NLR K-means iteration (GEM iteration): thin Python binding over libgemnlr.so.

Every step of the method runs in the CUDA library behind the C ABI declared in
include/gem_nlr.h; this package only marshals arguments.  There is no CPU fallback: loading
fails loudly if the library has not been built.
"""
from .binding import (  # noqa: F401
    GemNlr,
    IterInfo,
    Params,
    lib,
    library_path,
    run_host,
    workspace_bytes,
    paper_storage_bytes,
    host_job_device_bytes,
    column_sums_static,
    E_TIMEOUT, E_TOO_LARGE, STATIC_MAX_R,
    OK, CONVERGED, ITER_CAP, E_INVALID, E_CUDA, E_WORKSPACE, E_BREAKDOWN, E_NONFINITE, E_NOT_READY,
)
