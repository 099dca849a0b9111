"""Pins for the planner oracle: cover/disjointness, exact pair totals, the closed-form
balance of zigzag partitions (tests/golden/planner_balance.txt) and per-pair brute force
for the causal tile classes."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden_rows():
    rows = []
    for line in open(os.path.join(GOLDEN, "planner_balance.txt")):
        if line.strip() and not line.startswith("#"):
            rows.append(tuple(int(x) for x in line.split()))
    return rows


@pytest.mark.parametrize("S,P,align,pairs", _golden_rows())
def test_zigzag_balance_closed_form(S, P, align, pairs):
    plan = oracle.plan_partitions(S, P, 0, align, 128, 128, True, tiles=False)
    assert plan["pairs"] == [pairs] * P
    b = S // (2 * P)
    for p in range(P):
        assert plan["parts"][p] == [(p * b, (p + 1) * b), ((2 * P - 1 - p) * b, (2 * P - p) * b)]


@pytest.mark.parametrize("S,P,align", [(1, 1, 1), (1, 4, 128), (127, 2, 128), (1000, 3, 128), (1025, 4, 64),
                                       (4097, 8, 128), (300, 16, 16), (0, 2, 8)])
def test_partitions_are_a_disjoint_cover_with_exact_pair_total(S, P, align):
    plan = oracle.plan_partitions(S, P, 0, align, 64, 64, True, tiles=False)
    bounds = plan["bounds"]
    assert len(bounds) == 2 * P + 1 and bounds[0] == 0 and bounds[-1] == S
    assert all(bounds[i] <= bounds[i + 1] for i in range(2 * P))
    assert all(b % align == 0 or b == S for b in bounds)
    owner = np.full(S, -1)
    for p, ivs in enumerate(plan["parts"]):
        for lo, hi in ivs:
            assert (owner[lo:hi] == -1).all()
            owner[lo:hi] = p
    assert (owner >= 0).all()
    assert sum(plan["pairs"]) == S * (S + 1) // 2
    # per-pair brute force of one partition's count
    p = P // 2
    keys = [j for lo, hi in plan["parts"][p] for j in range(lo, hi)]
    if S <= 1100:
        assert plan["pairs"][p] == sum(1 for i in range(S) for j in keys if j <= i)
    nc = oracle.plan_partitions(S, P, 0, align, 64, 64, False, tiles=False)
    assert sum(nc["pairs"]) == S * S


@pytest.mark.parametrize("S,C", [(10, 3), (8192, 8192), (131072, 8192), (5, 100), (7, 0)])
def test_chunks_tile_the_rows(S, C):
    plan = oracle.plan_partitions(S, 1, C, 1, 128, 128, True, tiles=False)
    pos = 0
    for start, n in plan["chunks"]:
        assert start == pos and n > 0 and (C <= 0 or n <= C)
        pos += n
    assert pos == S
    if C > 0:
        assert len(plan["chunks"]) == -(-S // C)
        assert all(n == C for _, n in plan["chunks"][:-1])


@pytest.mark.parametrize("S,bm,bn", [(1024, 128, 128), (300, 64, 128), (257, 128, 64), (96, 32, 32), (5, 4, 2)])
def test_tile_classes_match_per_pair_brute_force(S, bm, bn):
    plan = oracle.plan_partitions(S, 1, 0, 1, bm, bn, True)
    vis = np.tril(np.ones((S, S), dtype=bool))      # vis[i, j] = key j visible to query i
    tc = plan["tile_class"]
    assert tc.shape == (-(-S // bm), -(-S // bn))
    for a in range(tc.shape[0]):
        for b in range(tc.shape[1]):
            blk = vis[a * bm:(a + 1) * bm, b * bn:(b + 1) * bn]
            want = oracle.FULL if blk.all() else (oracle.SKIP if not blk.any() else oracle.PARTIAL)
            assert tc[a, b] == want
    nc = oracle.plan_partitions(S, 1, 0, 1, bm, bn, False)["tile_class"]
    assert (nc == oracle.FULL).all()


def test_square_tiles_have_one_partial_tile_per_row_of_tiles():
    plan = oracle.plan_partitions(2048, 1, 0, 128, 128, 128, True)
    tc = plan["tile_class"]
    n = 16
    assert (tc == oracle.PARTIAL).sum() == n
    assert (tc == oracle.FULL).sum() == n * (n - 1) // 2
    assert (tc == oracle.SKIP).sum() == n * (n - 1) // 2


def test_kv_prefix_cuts_partition_intervals():
    assert oracle.partition_intervals(1024, 4, 0, 128) == [(0, 128), (896, 1024)]
    assert oracle.partition_intervals(1024, 4, 0, 128, kv_len=900) == [(0, 128), (896, 900)]
    assert oracle.partition_intervals(1024, 4, 0, 128, kv_len=512) == [(0, 128)]
    assert oracle.partition_intervals(1024, 1, 0, 128, kv_len=512) == [(0, 512)]
