"""CPU oracle for the TAOT planner.  TEST INFRASTRUCTURE ONLY -- never imported by the product.

`taot_oracle.c` holds the arithmetic; this module compiles it with gcc and wraps it with
numpy in/out.  Only tests, the smoke check and the benchmark's CPU-baseline leg import it.
"""
from .binding import (  # noqa: F401
    build,
    histogram,
    excess_spare,
    sinkhorn,
    sinkhorn_gibbs,
    default_preference,
    spill,
    match,
    auction,
    assign,
    plan_layers,
    report,
    dispatch,
    REPORT_INTS,
    REPORT_REALS,
)
