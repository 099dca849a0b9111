"""Section 5.3's SP strategy cost model: the oracle against a hand-worked example, limiting
cases and a brute-force argmin; the library against the oracle."""
import itertools
import os

import pytest

import oracle
from paper_2409_15104_b200 import binding

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "sp_volumes_worked.txt")
ORDER = [("megatron", "megatron"), ("megatron", "ulysses"), ("ulysses", "megatron"), ("ulysses", "ulysses")]


def test_oracle_volumes_match_the_hand_worked_example():
    want = [int(x) for line in open(GOLDEN) if line.strip() and not line.startswith("#") for x in line.split()]
    v = oracle.sp_volumes(2, 4, 2, 1, 2, 2, 4)
    got = [v[("attn", "megatron")][0], v[("attn", "megatron")][1], v[("attn", "ulysses")][0], v[("attn", "ulysses")][1],
           v[("mlp", "megatron")][0], v[("mlp", "megatron")][1], v[("mlp", "ulysses")][0], v[("mlp", "ulysses")][1]]
    assert got == want


def test_oracle_limiting_cases():
    # no tensor parallelism: Megatron SP moves nothing and no parameters travel
    v = oracle.sp_volumes(1000, 4096, 32, 8, 128, 1, 8)
    assert v[("attn", "megatron")][0] == 0 and v[("mlp", "megatron")][0] == 0 and v[("mlp", "ulysses")][0] == 0
    assert v[("attn", "ulysses")][0] == 2 * 1000 * 40 * 128 * 7
    # one GPU per node and no TP: nothing to exchange anywhere, and both strategies compute the same
    v = oracle.sp_volumes(1000, 4096, 32, 8, 128, 1, 1)
    assert all(c == 0 for c, _ in v.values())
    assert v[("attn", "megatron")][1] == v[("attn", "ulysses")][1]
    # attention term is quadratic in the segment length, the linear terms are linear
    a = oracle.sp_volumes(1000, 64, 4, 4, 16, 2, 2)[("attn", "megatron")][1]
    b = oracle.sp_volumes(2000, 64, 4, 4, 16, 2, 2)[("attn", "megatron")][1]
    lin = 2 * 1000 * 64 * 8 * 16 // 2 + 2 * 1000 * 64 * 64
    assert b - 2 * lin == 4 * (a - lin)


CASES = [
    (131072 // 8, 4096, 32, 8, 128, 1, 8), (500000 // 8, 8192, 64, 8, 128, 4, 8), (100000 // 8, 7168, 56, 8, 128, 4, 8),
    (2, 4, 2, 1, 2, 2, 4), (512, 4096, 32, 8, 128, 8, 8), (64, 1024, 8, 8, 128, 2, 2), (1 << 20, 4096, 32, 8, 128, 4, 8),
]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("bw,flops", [(900e9 * 8, 1.4e15), (50e9, 1.4e15), (7.2e12, 3e14)])
def test_library_matches_the_oracle(case, bw, flops):
    got = binding.pec_select_sp(*case, elem_bytes=2.0, node_bw=bw, gpu_flops=flops)
    vols = oracle.sp_volumes(*case)
    best, times = oracle.select_sp(*case, 2, bw, flops)
    for si, stage in enumerate(("attn", "mlp")):
        for ti, strat in enumerate(("megatron", "ulysses")):
            assert got["comm"][si][ti] == pytest.approx(float(vols[(stage, strat)][0]), rel=1e-12)
            assert got["comp"][si][ti] == pytest.approx(float(vols[(stage, strat)][1]), rel=1e-12)
    for i, combo in enumerate(ORDER):
        assert got["seconds"][i] == pytest.approx(float(times[combo]), rel=1e-12)
    # brute-force argmin over the four combinations; near-ties may legitimately differ in the last bit
    chosen = ORDER[2 * got["attn_strategy"] + got["mlp_strategy"]]
    assert float(times[chosen]) <= float(min(times.values())) * (1 + 1e-12)
    if all(abs(float(times[c]) - float(times[best])) > 1e-9 * float(times[best]) for c in ORDER if c != best):
        assert chosen == best


def test_long_segments_on_a_slow_link_prefer_less_traffic():
    """With T > 1 and a slow node link, the strategy moving fewer bytes wins each stage."""
    case = (65536, 8192, 64, 8, 128, 4, 8)
    got = binding.pec_select_sp(*case, elem_bytes=2.0, node_bw=1e9, gpu_flops=1e18)
    vols = oracle.sp_volumes(*case)
    for si, stage in enumerate(("attn", "mlp")):
        fewer = 0 if vols[(stage, "megatron")][0] <= vols[(stage, "ulysses")][0] else 1
        assert (got["attn_strategy"], got["mlp_strategy"])[si] == fewer


def test_bad_inputs_are_rejected():
    import ctypes
    lib = binding.load()
    out = binding.pec_sp_choice()
    ok = binding.pec_sp_inputs(10, 10, 2, 2, 4, 1, 1, 2, 1, 1)
    assert lib.pec_select_sp(ctypes.byref(ok), ctypes.byref(out)) == 0
    assert lib.pec_select_sp(None, ctypes.byref(out)) == -1
    for field, val in [("s", 0), ("T", 0.5), ("G", 0), ("node_bw", 0), ("gpu_flops", -1), ("d_h", float("nan"))]:
        bad = binding.pec_sp_inputs(10, 10, 2, 2, 4, 1, 1, 2, 1, 1)
        setattr(bad, field, val)
        assert lib.pec_select_sp(ctypes.byref(bad), ctypes.byref(out)) == -1, field
