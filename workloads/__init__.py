"""Seeded synthetic inputs for the TAOT planner (routing tables, topology costs, rank loads).

This package only *draws inputs*.  It holds none of the planner's arithmetic (no
histogram, no excess/spare, no Sinkhorn, no matching): both the CPU oracle's tests and the
CUDA path's tests/bench take their inputs from here and nothing else is shared between
them.  All generators are counter-based (a hash of (seed, layer, token, expert)), written
with integer tensor ops so the same call works on a CPU or a CUDA device.
"""
from .configs import PlannerConfig, CONFIGS, get_config, sweep_cells  # noqa: F401
from .generate import (  # noqa: F401
    cost_matrix,
    expert_to_rank,
    zipf_exponents,
    routing_topk,
    sweep_rank_loads,
    uniform01,
)
