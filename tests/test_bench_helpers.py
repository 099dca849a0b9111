"""CPU checks of the arithmetic bench.py reports with: exact merge bytes and the stored-counter bookkeeping."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench
import oracle


def test_merge_bytes_count_only_rows_that_hold_a_partial():
    """Brute force over (row, part): a part's row is live when it can see one of the part's keys (causal),
    i.e. from the part's first key on; live rows cost 516 bytes per head, empty ones their 4-byte LSE."""
    S, P, hq, align = 2048, 4, 3, 64
    plan = oracle.plan_partitions(S, P, 0, align, 128, 128, True, tiles=False)
    want = 0
    for p in range(P):
        first_key = min(lo for lo, hi in plan["parts"][p] if hi > lo)
        for row in range(S):
            want += hq * (516 if row >= first_key else 4)
    want += S * hq * 260
    assert bench.merge_bytes_exact(S, hq, plan["bounds"], range(P), True) == want
    assert bench.merge_bytes_exact(S, hq, plan["bounds"], range(P), False) == want + S * hq * 256


def test_stored_counters_are_tied_to_the_kernel_sources():
    rec = bench.stored_counters("c3")
    assert rec is not None and rec["captured_offline"] and rec["dram_bytes_per_launch"] > 0
    assert rec["stale"] == (rec["kernel_source_hash_at_capture"] != bench.kernel_source_hash())
    assert bench.stored_counters("no such workload") is None
