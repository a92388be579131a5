"""Seeded synthetic workloads for the batched elastic scheduling round.

This package only *draws inputs*: action records (pool, unit, level mask, runtime
parameters, arrivals) and pool descriptions.  It contains none of the scheduling
method's arithmetic (no duration model, no capacity test, no selection), so the
CPU oracle and the CUDA library can both be fed from it without sharing any of
the method's code.

Random numbers are counter based: every draw is splitmix64 applied to a key made
of (base seed + scenario id, action index, field id), so any scenario can be
regenerated alone and chunks of scenarios can be generated independently.
"""
from .generator import (  # noqa: F401
    POOL_CPU,
    POOL_GPU,
    POOL_API,
    GANG,
    Pool,
    Workload,
    CONFIGS,
    make_workload,
    generate,
    random_round,
    contiguous_replica_round,
    add_side_costs,
    add_trajectories,
    ablation_sweep,
)
