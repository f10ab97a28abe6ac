"""B200-native S2D2 decode step: thin Python binding over the C ABI in
include/s2d2.h.  Importing the package does not load the CUDA library; creating
an ``Engine`` does, and fails loudly if the library is missing."""
from .binding import (  # noqa: F401
    DraftStats,
    Engine,
    RoutePolicy,
    S2D2Error,
    StepResult,
    gemm_bf16_noalloc,
    library_path,
    load_library,
)
