"""CPU-only checks of the library's host side: exported symbols, planner parity with the
oracle (bit-exact), and argument validation (no kernel is launched by these calls)."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2409_15104_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    lib = binding.load()
    header = open(os.path.join(ROOT, "include", "pec.h")).read()
    declared = set(re.findall(r"\b(pec_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


PLAN_CASES = [
    (1024, 4, 0, 128, 128, 128, True), (32768, 8, 0, 128, 128, 128, True), (131072, 1, 8192, 128, 128, 128, True),
    (1000, 3, 64, 128, 128, 128, True), (1, 1, 1, 1, 1, 1, True), (0, 2, 0, 8, 16, 16, True),
    (4097, 8, 1000, 128, 64, 128, True), (300, 16, 7, 16, 32, 64, False), (8191, 5, 0, 1, 128, 128, True),
    (127, 2, 0, 128, 128, 128, True),
]


@pytest.mark.parametrize("case", PLAN_CASES)
def test_planner_matches_oracle_bit_exactly(case):
    S, P, C, align, bm, bn, causal = case
    tiles = S <= 40000
    got = binding.pec_plan_partitions(S, P, C, align, bm, bn, causal, tiles=tiles)
    want = oracle.plan_partitions(S, P, C, align, bm, bn, causal, tiles=tiles)
    assert got["bounds"] == want["bounds"]
    assert got["parts"] == want["parts"]
    assert got["pairs"] == want["pairs"]
    assert got["chunks"] == want["chunks"]
    assert (got["nq_tiles"], got["nk_tiles"]) == (want["nq_tiles"], want["nk_tiles"])
    if tiles:
        assert np.array_equal(got["tile_class"], want["tile_class"])


def test_planner_largest_config_pairs():
    got = binding.pec_plan_partitions(262144, 16, 0, 128, 128, 128, True, tiles=False)
    assert got["pairs"] == [8192 * 262145] * 16            # closed form b*(S+1)
    assert got["nq_tiles"] == 2048 and got["nk_tiles"] == 2048


def test_planner_rejects_bad_arguments_and_small_arrays():
    lib = binding.load()
    plan = binding.pec_plan()
    assert lib.pec_plan_partitions(-1, 1, 0, 1, 1, 1, 1, ctypes.byref(plan)) == -1
    assert lib.pec_plan_partitions(10, 0, 0, 1, 1, 1, 1, ctypes.byref(plan)) == -1
    assert lib.pec_plan_partitions(10, 1, 0, 0, 1, 1, 1, ctypes.byref(plan)) == -1
    assert lib.pec_plan_partitions(10, 1, 0, 1, 1, 1, 1, None) == -1
    assert "plan is NULL" in binding.pec_last_error()
    buf = (ctypes.c_int64 * 2)()
    plan.bounds, plan.bounds_cap = buf, 2
    assert lib.pec_plan_partitions(10, 2, 0, 1, 1, 1, 1, ctypes.byref(plan)) == -7
    assert plan.n_bounds == 5


def _args(**over):
    a = binding.pec_attn_args()
    a.q = a.k = a.v = a.o = a.lse = 4096          # never dereferenced: validation fails first
    a.status = 4096
    a.q_stride_t, a.q_stride_h = 8 * 128, 128
    a.k_stride_t, a.k_stride_h = 8 * 128, 128
    a.v_stride_t, a.v_stride_h = 8 * 128, 128
    a.in_dtype, a.o_dtype = binding.PEC_BF16, binding.PEC_BF16
    a.Hq, a.Hkv, a.D = 8, 8, 128
    a.B, a.seq_len, a.chunk_start, a.chunk_len, a.kv_len = 1, 256, 0, 256, 256
    a.part_id, a.num_parts, a.part_align, a.causal = 0, 1, 128, 1
    for k, v in over.items():
        setattr(a, k, v)
    return a


@pytest.mark.parametrize("over,code", [
    (dict(q=None), -1), (dict(D=64), -2), (dict(Hq=6, Hkv=4), -1), (dict(in_dtype=7), -2),
    (dict(in_dtype=binding.PEC_F32, o_dtype=binding.PEC_BF16), -2), (dict(causal=2), -1),
    (dict(chunk_start=200, chunk_len=100), -1), (dict(kv_len=100), -1), (dict(part_id=2, num_parts=2), -1),
    (dict(q=4100), -3), (dict(k_stride_t=8 * 128 + 4), -3), (dict(q_stride_h=64), -1),
    (dict(cu_seqlens=4096, B=2, chunk_len=100), -1), (dict(softmax_scale=float("nan")), -1),
    (dict(part_align=0), -1),
    (dict(acc_o=8192), -1),                                            # incoming state without its LSE
    (dict(acc_o=4096, acc_lse=8192, o_dtype=binding.PEC_F32), -1),    # o is the state's buffer, lse is not
    (dict(acc_o=4096, acc_lse=4096), -1),                              # in-place merge needs fp32 output
    (dict(acc_o=8196, acc_lse=12288), -3),
    (dict(q_num_parts=4, q_part_id=4), -1), (dict(q_num_parts=2, q_part_id=-1), -1),
    (dict(cu_seqlens=4096, B=2, q_num_parts=2), -1),                   # query partitions are for single requests
    (dict(status=None), -1),                                           # bf16 inputs need the status word
    (dict(overlap_previous=2), -1),
    (dict(worklist=4096, n_items=3), -1),                              # a work-list without cu_seqlens
    (dict(cu_seqlens=4096, B=2, worklist=4096, n_items=3, worklist_block_m=64), -1),   # built for the other kernel's tiles
    (dict(cu_seqlens=4096, B=2, worklist=4100, n_items=3, worklist_block_m=256), -1),
])
def test_prefill_attn_validates_on_the_host(over, code):
    lib = binding.load()
    a = _args(**over)
    assert lib.pec_prefill_attn(ctypes.byref(a), None) == code
    assert binding.pec_last_error()
    assert lib.pec_prefill_attn(None, None) == -1


def test_merge_validates_on_the_host():
    lib = binding.load()
    f = lib.pec_attn_merge
    ok = [4096, 8192, 12288, 16384, 20480, 24576]
    assert f(None, *ok[1:], 4, 2, 128, 2, 2, None) == -1
    assert f(*ok, 4, 2, 64, 2, 2, None) == -2
    assert f(*ok, 4, 2, 128, 1, 2, None) == -2
    assert f(*ok, -1, 2, 128, 2, 2, None) == -1
    assert f(4100, *ok[1:], 4, 2, 128, 2, 2, None) == -3
    assert f(ok[0], ok[1], ok[2], ok[3], ok[0], ok[5], 4, 2, 128, 2, 2, None) == -1   # o aliased, lse not
    assert f(ok[0], ok[1], ok[2], ok[3], ok[2], ok[3], 4, 2, 128, 2, 2, None) == -1   # aliasing side b
    assert f(*ok, 0, 2, 128, 2, 2, None) == 0                                          # nothing to do


def test_merge_n_validates_on_the_host():
    lib = binding.load()
    f = lib.pec_attn_merge_n

    def ptrs(vals):
        return (ctypes.c_void_p * len(vals))(*vals)

    o3, l3 = ptrs([4096, 8192, 12288]), ptrs([16384, 20480, 24576])
    assert f(o3, l3, 3, 32768, 36864, 0, 2, 128, 2, 2, None) == 0            # nothing to do
    assert f(o3, l3, 1, 32768, 36864, 4, 2, 128, 2, 2, None) == -1           # n too small
    assert f(o3, l3, 17, 32768, 36864, 4, 2, 128, 2, 2, None) == -1          # n too large
    assert f(None, l3, 3, 32768, 36864, 4, 2, 128, 2, 2, None) == -1
    assert f(o3, l3, 3, 32768, 36864, 4, 2, 64, 2, 2, None) == -2
    assert f(o3, l3, 3, 32768, 36864, 4, 2, 128, 1, 2, None) == -2
    assert f(ptrs([4100, 8192, 12288]), l3, 3, 32768, 36864, 4, 2, 128, 2, 2, None) == -3
    assert f(o3, l3, 3, 8192, 20480, 4, 2, 128, 2, 2, None) == -1            # aliasing part 1
    assert f(o3, l3, 3, 4096, 36864, 4, 2, 128, 2, 2, None) == -1            # o aliases part 0, lse does not
    assert f(o3, l3, 3, 4096, 16384, 4, 2, 128, 2, 1, None) == -1            # aliasing with bf16 output
    assert "alias" in binding.pec_last_error()


def test_decode_validates_on_the_host_and_sizes_its_workspace():
    lib = binding.load()
    a = binding.pec_decode_args()
    a.q = a.k = a.v = a.o = a.lse = a.status = 4096
    a.q_stride_h = 128
    a.k_stride_t = a.v_stride_t = 8 * 128
    a.k_stride_h = a.v_stride_h = 128
    a.o_dtype, a.Hq, a.Hkv, a.D = binding.PEC_F32, 32, 8, 128
    a.kv_lo, a.kv_hi, a.num_splits = 0, 100000, 10
    need = lib.pec_decode_workspace_size(ctypes.byref(a))
    # 10 slices of ceil(10000/128)*128 = 10112 keys -> still 10 slices; 516 bytes per (slice, head)
    assert need == 10 * 32 * 516
    assert lib.pec_decode_attn(ctypes.byref(a), None) == -4            # no workspace given
    a.workspace, a.workspace_bytes = 4096, need - 1
    assert lib.pec_decode_attn(ctypes.byref(a), None) == -4
    for field, val, code in [("D", 64, -2), ("Hq", 30, -1), ("kv_hi", -1, -1), ("num_splits", 5000, -1),
                             ("q", 4100, -3), ("k_stride_t", 1028, -3), ("status", None, -1), ("o_dtype", 9, -2)]:
        old = getattr(a, field)
        setattr(a, field, val)
        assert lib.pec_decode_attn(ctypes.byref(a), None) == code, field
        assert lib.pec_decode_workspace_size(ctypes.byref(a)) == 0
        setattr(a, field, old)


def test_linear_rope_and_table_validate_on_the_host():
    lib = binding.load()
    ok = dict(x=4096, xs=64, w=8192, ws=64, y=12288, ys=256, M=10, N=256, K=64, t=65536, npos=100, pos=None, pos0=0,
              rot=128, st=16384)

    def call(**over):
        a = {**ok, **over}
        return lib.pec_linear_rope(a["x"], a["xs"], a["w"], a["ws"], a["y"], a["ys"], a["M"], a["N"], a["K"], a["t"],
                                   a["npos"], a["pos"], a["pos0"], a["rot"], a["st"], None)

    assert call(M=0) == 0
    assert call(t=None) == -1 and call(npos=0) == -1 and call(x=None) == -1
    assert call(rot=384) == -1 and call(rot=-128) == -1 and call(pos0=91) == -1 and call(pos0=-1) == -1
    assert call(rot=64) == -2 and call(N=260, ys=264) == -2
    assert call(t=65540) == -3 and call(pos=2050) == -3
    assert lib.pec_rope_table_floats(0) == 8192 and lib.pec_rope_table_floats(64) == 8192 + 128
    assert lib.pec_rope_table_floats(65) == 8192 + 256 and lib.pec_rope_table_floats(-1) == 0
    assert lib.pec_rope_table(500000.0, 10, 64, 4096, None) == -2
    assert lib.pec_rope_table(0.0, 10, 128, 4096, None) == -1 and lib.pec_rope_table(1e4, 10, 128, None, None) == -1
    assert lib.pec_rope_table(1e4, 10, 128, 4100, None) == -3


def test_linear_merged_validates_on_the_host():
    import ctypes
    f = binding.load().pec_linear_merged

    def call(o=(4096, 8192), l=(256, 512), n=2, rows=10, Hq=1, D=128, w=16384, ws=128, y=32768, ys=32, N=32, st=65536):
        op = (ctypes.c_void_p * max(len(o), 1))(*o)
        lp = (ctypes.c_void_p * max(len(l), 1))(*l)
        return f(op, lp, n, rows, Hq, D, w, ws, y, ys, N, st, None)

    assert call(rows=0) == 0
    assert call(n=0) == -1 and call(n=9, o=(4096,) * 9, l=(256,) * 9) == -1 and call(st=None) == -1 and call(w=None) == -1
    assert call(o=(4096, None)) == -1 and call(rows=-1) == -1 and call(Hq=0) == -1 and call(N=0) == -1
    assert call(D=64) == -2 and call(N=36) == -2
    assert call(ws=64) == -1 and call(ys=16) == -1
    assert call(o=(4100, 8192)) == -3 and call(ws=132) == -3 and call(y=32772) == -3


def test_linear_validates_on_the_host():
    f = binding.load().pec_linear
    ok = dict(x=4096, xs=64, w=8192, ws=64, y=12288, ys=32, M=10, N=32, K=64, st=16384)

    def call(**over):
        a = {**ok, **over}
        return f(a["x"], a["xs"], a["w"], a["ws"], a["y"], a["ys"], a["M"], a["N"], a["K"], a["st"], None)

    assert call(M=0) == 0
    assert call(x=None) == -1 and call(st=None) == -1 and call(M=-1) == -1 and call(N=0) == -1
    assert call(N=30) == -2 and call(K=60, xs=64) == -2
    assert call(xs=32) == -1 and call(ys=16) == -1
    assert call(x=4100) == -3 and call(ws=68) == -3
