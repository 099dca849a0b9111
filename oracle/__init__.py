"""fp64 CPU oracle for partial causal attention, its merge and the partition planner.

Test infrastructure only: nothing in the GPU library imports this package, and this
package imports nothing from the GPU library.
"""
from .reference import (  # noqa: F401
    attn_rows,
    prefill_attn,
    varlen_attn,
    merge,
    merge_n,
    sp_volumes,
    select_sp,
    linear,
    rope,
    linear_rope,
    plan_partitions,
    plan_worklist,
    partition_rows,
    plan_ring,
    ring_segments,
    balance_batches,
    partition_intervals,
    oracle_threads,
    SKIP,
    PARTIAL,
    FULL,
)
