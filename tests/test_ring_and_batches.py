"""Pins for the ring-attention work plan and the token-balanced batch builder (oracle side), and
bit-exact parity of the library's host code with the oracle.  No GPU is needed."""
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_2409_15104_b200 import binding

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
LAYOUTS = {"zigzag": binding.PEC_LAYOUT_ZIGZAG, "contiguous": binding.PEC_LAYOUT_CONTIGUOUS}


def _golden_rows():
    rows = []
    for line in open(os.path.join(GOLDEN, "ring_step_pairs.txt")):
        if line.strip() and not line.startswith("#"):
            rows.append(tuple(int(x) for x in line.split()))
    return rows


def _closed_form_plan(S, P, align, layout):
    """Same quantity from per-interval closed forms instead of row loops (large S)."""
    seg = oracle.ring_segments(S, P, align, layout)

    def count(a, b, c, d):
        # rows [a, b) against keys [c, d), causal: row i sees min(d, i + 1) - c keys when positive
        idx = np.arange(a, b, dtype=np.int64)
        return int(np.clip(np.minimum(d, idx + 1) - c, 0, None).sum())
    return [[sum(count(a, b, c, d) for a, b in seg[r] for c, d in seg[(r - t) % P]) for t in range(P)] for r in range(P)]


@pytest.mark.parametrize("S,P,align,z0,zt,c_first,c_last", _golden_rows())
def test_ring_plan_hand_worked_block_counts(S, P, align, z0, zt, c_first, c_last):
    pairs = _closed_form_plan(S, P, align, "zigzag") if S > 4096 else oracle.plan_ring(S, P, align, "zigzag", True)["pairs"]
    for r in range(P):
        assert pairs[r][0] == z0
        assert all(pairs[r][t] == zt for t in range(1, P))
    if S <= 4096:
        cont = oracle.plan_ring(S, P, align, "contiguous", True)
        assert cont["rank_total"][0] == c_first and cont["rank_total"][-1] == c_last
        # the imbalance the zigzag pairing removes
        assert 0.95 * (2 * P - 1) < cont["rank_total"][-1] / cont["rank_total"][0] < 2 * P - 1
        # a contiguous ring step is as slow as a full block although most ranks then have less or nothing to do
        c = S // P
        assert cont["step_max"][1:] == [c * c] * (P - 1)
    # the library, at every size
    got = binding.pec_plan_ring(S, P, align, binding.PEC_LAYOUT_ZIGZAG, True)
    assert got["pairs"] == [[z0] + [zt] * (P - 1)] * P
    got = binding.pec_plan_ring(S, P, align, binding.PEC_LAYOUT_CONTIGUOUS, True)
    assert got["rank_total"][0] == c_first and got["rank_total"][-1] == c_last


@pytest.mark.parametrize("layout", ["zigzag", "contiguous"])
@pytest.mark.parametrize("S,P,align", [(1, 1, 1), (7, 2, 1), (13, 3, 2), (40, 4, 4), (33, 5, 8), (0, 2, 4)])
def test_ring_plan_against_explicit_pair_enumeration(S, P, align, layout):
    seg = oracle.ring_segments(S, P, align, layout)
    owner = {}
    for r, ivs in enumerate(seg):
        for lo, hi in ivs:
            for i in range(lo, hi):
                assert i not in owner
                owner[i] = r
    assert sorted(owner) == list(range(S))                       # segments are a disjoint cover
    for causal in (True, False):
        want = [[0] * P for _ in range(P)]
        for i in range(S):
            for j in range(S):
                if j <= i or not causal:
                    want[owner[i]][(owner[i] - owner[j]) % P] += 1
        plan = oracle.plan_ring(S, P, align, layout, causal)
        assert plan["pairs"] == want
        total = S * (S + 1) // 2 if causal else S * S
        assert sum(plan["rank_total"]) == total
        assert binding.pec_plan_ring(S, P, align, LAYOUTS[layout], causal) == plan


@pytest.mark.parametrize("S,P,align", [(1000, 3, 128), (4097, 8, 128), (300, 16, 16), (2048, 4, 128), (777, 7, 1)])
def test_ring_plan_library_matches_oracle_on_ragged_sizes(S, P, align):
    for layout, code in LAYOUTS.items():
        for causal in (True, False):
            assert binding.pec_plan_ring(S, P, align, code, causal) == oracle.plan_ring(S, P, align, layout, causal)


def test_ring_plan_rejects_bad_arguments():
    for args in [(-1, 2, 128, 0, 1), (10, 0, 128, 0, 1), (10, 2, 0, 0, 1), (10, 2, 128, 7, 1)]:
        with pytest.raises(binding.PecError):
            binding.pec_plan_ring(*args[:3], layout=args[3], causal=bool(args[4]))


# ------------------------------------------------------------------ token-balanced batches
def _best_possible_max(lengths, replicas):
    best = None
    for assign in itertools.product(range(replicas), repeat=len(lengths)):
        tok = [0] * replicas
        for i, r in enumerate(assign):
            tok[r] += lengths[i]
        best = max(tok) if best is None else min(best, max(tok))
    return best


def test_balance_hand_worked_example():
    # longest first: 9 -> r0, 7 -> r1, 6 -> r1 (7 < 9), 5 -> r0 (9 < 13), 5 -> r1 (13 < 14), 1 -> r0
    assign, tokens = oracle.balance_batches([5, 9, 1, 7, 6, 5], 2)
    assert assign == [0, 0, 0, 1, 1, 1] and tokens == [15, 18]
    # equal lengths go in index order to the lowest replica id with the fewest tokens
    assert oracle.balance_batches([4, 4, 4, 4, 4], 3) == ([0, 1, 2, 0, 1], [8, 8, 4])
    assert oracle.balance_batches([], 3) == ([], [0, 0, 0])
    assert oracle.balance_batches([3, 0, 2], 1) == ([0, 0, 0], [5])


@pytest.mark.parametrize("seed", range(12))
def test_balance_within_the_longest_first_bound_of_the_optimum(seed):
    g = np.random.Generator(np.random.Philox(key=100 + seed))
    n, replicas = int(g.integers(1, 9)), int(g.integers(1, 4))
    lengths = [int(x) for x in g.integers(0, 50, size=n)]
    assign, tokens = oracle.balance_batches(lengths, replicas)
    assert sorted(set(assign)) <= list(range(replicas))
    for r in range(replicas):
        assert tokens[r] == sum(lengths[i] for i in range(n) if assign[i] == r)
    best = _best_possible_max(lengths, replicas)
    assert best <= max(tokens) <= best * (4 / 3 - 1 / (3 * replicas)) + 1e-9
    assert max(tokens) - min(tokens) <= max(lengths)             # no replica waits longer than one request
    assert binding.pec_balance_batches(lengths, replicas) == (assign, tokens)


def test_balance_library_matches_oracle_on_the_short_request_length_mix():
    from paper_2409_15104_b200 import workloads
    lengths = workloads.short_lengths(workloads.BASE_SEED + 2, 64)
    for replicas in (1, 2, 4, 8):
        got = binding.pec_balance_batches(lengths, replicas)
        assert got == oracle.balance_batches(lengths, replicas)
        assert sum(got[1]) == sum(lengths)
    with pytest.raises(binding.PecError):
        binding.pec_balance_batches([3, -1], 2)
    with pytest.raises(binding.PecError):
        binding.pec_balance_batches([3], 0)
