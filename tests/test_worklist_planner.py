"""Pins of the packed-batch work-list rule (Section 5.2's short-request batches) and parity of the
library's planner with the oracle's.  CPU only."""
import os

import numpy as np
import pytest

import oracle
from paper_2409_15104_b200 import binding, workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _brute_weight(pos0, n, L, block_n, causal):
    """Key tiles of the request that hold at least one (query, key) pair the mask lets through."""
    tiles = set()
    for i in range(pos0, pos0 + n):
        for j in range(L):
            if j <= i or not causal:
                tiles.add(j // block_n)
    return len(tiles)


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("lens,bm,bn", [([5], 4, 2), ([9, 0, 3, 17], 4, 4), ([1, 1, 1], 8, 8), ([33, 7, 64, 2], 16, 8), ([], 4, 4)])
def test_worklist_covers_every_row_once_heaviest_first(lens, bm, bn, causal):
    cu = workloads.cu_seqlens(lens)
    items = oracle.plan_worklist(cu, bm, bn, causal)
    seen = np.zeros(cu[-1], dtype=np.int32)
    weights = []
    for start, pos0, n, L in items:
        b = cu.index(start) if lens else None
        assert 1 <= n <= bm and pos0 % bm == 0 and pos0 + n <= L
        assert n == bm or pos0 + n == L                     # only a request's last tile is ragged
        seen[start + pos0:start + pos0 + n] += 1
        weights.append(_brute_weight(pos0, n, L, bn, causal))
    assert (seen == 1).all()
    assert weights == sorted(weights, reverse=True)
    assert len(items) == sum(-(-L // bm) for L in lens)


def test_worklist_hand_worked_example():
    """tests/golden/worklist_worked.txt: requests of 5, 2 and 9 rows, tiles of 4 rows, key tiles of 2."""
    path = os.path.join(ROOT, "tests", "golden", "worklist_worked.txt")
    want = [tuple(int(x) for x in ln.split()) for ln in open(path) if ln.strip() and not ln.startswith("#")]
    assert oracle.plan_worklist([0, 5, 7, 16], 4, 2, True) == want


def test_worklist_ties_keep_request_then_position_order():
    items = oracle.plan_worklist(workloads.cu_seqlens([8, 8]), 4, 4, True)
    assert items == [(0, 4, 4, 8), (8, 4, 4, 8), (0, 0, 4, 8), (8, 0, 4, 8)]


@pytest.mark.parametrize("S,P,align,c0,n", [(64, 4, 8, 0, 64), (100, 3, 4, 17, 60), (50, 2, 1, 49, 1), (37, 5, 16, 0, 37)])
def test_partition_rows_split_the_chunk(S, P, align, c0, n):
    """The rows a ring rank keeps: over all ranks they give every row of the chunk exactly once, and each
    rank's rows are those of its two zigzag blocks, checked against the bounds formula written out here."""
    U = -(-S // align)
    bounds = [min(S, align * ((k * U) // (2 * P))) for k in range(2 * P + 1)]
    seen = []
    for p in range(P):
        rows = oracle.partition_rows(S, P, p, align, c0, n)
        want = [i for i in range(c0, c0 + n) if bounds[p] <= i < bounds[p + 1] or bounds[2 * P - 1 - p] <= i < bounds[2 * P - p]]
        assert rows == want
        seen += rows
    assert sorted(seen) == list(range(c0, c0 + n))


@pytest.mark.parametrize("seed", range(6))
def test_library_worklist_matches_oracle_bit_exactly(seed):
    g = np.random.Generator(np.random.Philox(key=4242 + seed))
    lens = [int(x) for x in g.integers(0, 1500, size=int(g.integers(1, 90)))]
    cu = workloads.cu_seqlens(lens)
    for bm, bn, causal in [(256, 128, True), (64, 128, True), (256, 128, False), (7, 3, True)]:
        got = binding.pec_plan_worklist(cu, bm, bn, causal)
        want = oracle.plan_worklist(cu, bm, bn, causal)
        assert [tuple(int(x) for x in row) for row in got] == want


def test_library_worklist_for_the_short_batch_configuration():
    wl = workloads.WORKLOADS["c2"]
    cu = workloads.cu_seqlens(workloads.short_lengths(wl.seed, wl.short_batch))
    got = binding.pec_plan_worklist(cu, binding.pec_worklist_block_m(wl.dtype), 128, True)
    want = oracle.plan_worklist(cu, 256, 128, True)
    assert [tuple(int(x) for x in row) for row in got] == want
    assert got[0][1] + got[0][2] == max(b - a for a, b in zip(cu, cu[1:]))     # the longest request's last tile leads


def test_library_worklist_rejects_bad_arguments():
    import ctypes
    lib = binding.load()
    n = ctypes.c_int64(0)
    cu = (ctypes.c_int32 * 3)(0, 5, 3)
    assert lib.pec_plan_worklist(cu, 2, 4, 4, 1, None, 0, ctypes.byref(n)) == -1          # decreasing
    cu = (ctypes.c_int32 * 3)(0, 5, 9)
    assert lib.pec_plan_worklist(None, 2, 4, 4, 1, None, 0, ctypes.byref(n)) == -1
    assert lib.pec_plan_worklist(cu, 2, 0, 4, 1, None, 0, ctypes.byref(n)) == -1
    assert lib.pec_plan_worklist(cu, 2, 4, 4, 1, None, 0, ctypes.byref(n)) == 0 and n.value == 3
    buf = (ctypes.c_int32 * 8)()
    assert lib.pec_plan_worklist(cu, 2, 4, 4, 1, buf, 2, ctypes.byref(n)) == -7
    assert lib.pec_worklist_block_m(binding.PEC_BF16) == 256 and lib.pec_worklist_block_m(binding.PEC_F32) == 64
    assert lib.pec_worklist_block_m(9) == 0
