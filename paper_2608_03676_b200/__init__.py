"""B200-native TAOT replica-placement planner: thin Python binding over libtaot.so.

Every step of the path runs in the CUDA library; this package only marshals torch device
tensors into the C ABI declared in include/taot.h.  There is no CPU fallback: importing the
binding without the compiled library raises.
"""
from .binding import (  # noqa: F401
    Planner,
    TaotError,
    TaotParams,
    INFO_BAD_INDEX,
    INFO_SINKHORN_CAP,
    INFO_NONFINITE,
    INFO_AUCTION_RESIDUAL,
    INFO_SUPPLY_SCALED,
    INFO_SINKHORN_SIZE,
    library_path,
    load_library,
    exported_symbols,
    histogram_static,
    STATIC_SCRATCH_BYTES,
    PLAN_LAUNCHES,
    PLAN_LAUNCHES_NO_HINT,
    ABLATE_HINT,
    ABLATE_TOPOLOGY,
    INFO_INTERNAL,
    ReportRow,
    measure_alu_peaks,
    measure_latencies,
    measure_round_latencies,
    PipelinedHostPlanner,
    StreamingHostPlanner,
    split_layers,
)
from .report import format_layer  # noqa: F401
