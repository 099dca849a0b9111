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


def test_gemm_roofline_takes_the_peak_that_matches_the_timed_region():
    peaks = {"bf16_burst": 1600.0, "bf16_sustained": 1400.0, "hbm": 6500.0, "source": "measured"}
    short = bench._gemm_roofline(1500.0, 40.0, peaks)                  # 40 ms timed: burst conditions
    long = bench._gemm_roofline(1300.0, 5000.0, peaks)                 # 5 s timed: at the power cap
    assert short["peak"] == 1600.0 and abs(short["frac"] - 1500.0 / 1600.0) < 1e-12
    assert long["peak"] == 1400.0 and abs(long["frac"] - 1300.0 / 1400.0) < 1e-12
    for r in (short, long):
        assert abs(r["frac_of_burst"] - r["achieved"] / 1600.0) < 1e-12 and abs(r["frac_of_sustained"] - r["achieved"] / 1400.0) < 1e-12


def test_the_stored_counters_of_the_headline_workload_are_current():
    """roofline.traffic of the bench line comes from profiles/attn_counters.txt and is nulled when the attention kernel's
    sources have changed since the capture: a change to those files must come with a new capture."""
    for name in ("c3", "c5"):
        assert not bench.stored_counters(name)["stale"], f"profiles/attn_counters.txt: the {name} capture is older than the kernel sources"
