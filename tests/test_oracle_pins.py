"""Pins for the fp64 attention/merge oracle against things other than itself:
brute force on tiny inputs, closed forms, a hand-worked case, a library routine
(torch scaled_dot_product_attention / logsumexp in fp64) and exact invariants."""
import math
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(shape, seed):
    g = np.random.Generator(np.random.Philox(key=seed))
    return g.standard_normal(shape).astype(np.float32)


def brute_force(q, k, v, q_pos, visible_keys, causal, scale):
    """Per-pair Python loops with an explicit 0/1 mask matrix (tiny shapes only)."""
    n, hq, d = q.shape
    nk, hkv, _ = k.shape
    g = hq // hkv
    mask = [[1 if (j in visible_keys and (not causal or j <= q_pos[i])) else 0
             for j in range(nk)] for i in range(n)]
    o = np.zeros((n, hq, d))
    lse = np.full((n, hq), -np.inf)
    for i in range(n):
        for h in range(hq):
            a = []
            for j in range(nk):
                if mask[i][j]:
                    s = 0.0
                    for c in range(d):
                        s += float(q[i, h, c]) * float(k[j, h // g, c])
                    a.append((j, s * scale))
            if not a:
                continue
            z = sum(math.exp(s) for _, s in a)
            for j, s in a:
                p = math.exp(s) / z
                for c in range(d):
                    o[i, h, c] += p * float(v[j, h // g, c])
            lse[i, h] = math.log(z)
    return o, lse


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("hq,hkv", [(2, 2), (4, 2), (4, 1)])
def test_brute_force_tiny(causal, hq, hkv):
    S, d = 8, 4
    q, k, v = _rand((S, hq, d), 1), _rand((S, hkv, d), 2), _rand((S, hkv, d), 3)
    pos = np.arange(S)
    for ivs in ([(0, 8)], [(0, 2), (6, 8)], [(2, 4), (4, 6)], [(3, 3)], [(5, 8)]):
        keys = {j for lo, hi in ivs for j in range(lo, hi)}
        o, lse = oracle.attn_rows(q, pos, k, v, ivs, causal, scale=0.5)
        ob, lb = brute_force(q, k, v, pos, keys, causal, 0.5)
        np.testing.assert_allclose(o, ob, rtol=0, atol=1e-13)
        assert np.array_equal(np.isneginf(lse), np.isneginf(lb))
        fin = ~np.isneginf(lb)
        np.testing.assert_allclose(lse[fin], lb[fin], rtol=0, atol=1e-13)
        assert (o[~fin] == 0).all()


def test_brute_force_query_positions_offset():
    """Rows given by position (a chunk in the middle of the request) see keys up to themselves."""
    S, d = 7, 3
    q, k, v = _rand((S, 2, d), 4), _rand((S, 1, d), 5), _rand((S, 1, d), 6)
    pos = np.array([5, 2, 6])
    o, lse = oracle.attn_rows(q[pos], pos, k, v, [(0, S)], True, scale=1.0)
    ob, lb = brute_force(q[pos], k, v, pos, set(range(S)), True, 1.0)
    np.testing.assert_allclose(o, ob, atol=1e-13)
    np.testing.assert_allclose(lse, lb, atol=1e-13)


@pytest.mark.parametrize("S,hq,hkv,d", [(257, 4, 2, 128), (64, 8, 8, 32), (300, 6, 2, 16)])
def test_matches_torch_sdpa_fp64(S, hq, hkv, d):
    """Library special case: causal SDPA and logsumexp in fp64 (textbook routines)."""
    q, k, v = _rand((S, hq, d), 11), _rand((S, hkv, d), 12), _rand((S, hkv, d), 13)
    o, lse = oracle.attn_rows(q, np.arange(S), k, v, [(0, S)], True)
    tq = torch.from_numpy(q).double().permute(1, 0, 2)[None]
    g = hq // hkv
    tk = torch.from_numpy(k).double().repeat_interleave(g, dim=1).permute(1, 0, 2)[None]
    tv = torch.from_numpy(v).double().repeat_interleave(g, dim=1).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    np.testing.assert_allclose(o, ref[0].permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)
    scores = torch.einsum("bhid,bhjd->bhij", tq, tk) / math.sqrt(d)
    scores = scores.masked_fill(torch.ones(S, S).triu(1).bool(), float("-inf"))
    ref_lse = torch.logsumexp(scores, dim=-1)[0].permute(1, 0).numpy()
    np.testing.assert_allclose(lse, ref_lse, rtol=0, atol=1e-12)


def test_noncausal_matches_torch_sdpa_fp64():
    S, hq, hkv, d = 96, 4, 4, 64
    q, k, v = _rand((S, hq, d), 21), _rand((S, hkv, d), 22), _rand((S, hkv, d), 23)
    o, _ = oracle.attn_rows(q, np.arange(S), k, v, [(0, S)], False)
    tq, tk, tv = (torch.from_numpy(x).double().permute(1, 0, 2)[None] for x in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)
    np.testing.assert_allclose(o, ref[0].permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)


def test_uniform_scores_give_prefix_mean_of_v():
    """Q = 0: every visible key has score 0, so O_i = mean(V[0..i]) and LSE_i = ln(i+1)."""
    S, h, d = 50, 2, 8
    q = np.zeros((S, h, d), np.float32)
    k, v = _rand((S, h, d), 31), _rand((S, h, d), 32)
    o, lse = oracle.attn_rows(q, np.arange(S), k, v, [(0, S)], True)
    want = np.cumsum(v.astype(np.float64), axis=0) / np.arange(1, S + 1)[:, None, None]
    np.testing.assert_allclose(o, want, atol=1e-13)
    np.testing.assert_allclose(lse, np.log(np.arange(1, S + 1))[:, None].repeat(h, 1), atol=1e-13)


def test_equal_keys_shift_lse_by_the_common_score():
    S, d = 20, 4
    q, v = _rand((S, 1, d), 41), _rand((S, 1, d), 42)
    k = np.tile(np.array([1.0, -2.0, 0.5, 0.25], np.float32), (S, 1, 1))
    o, lse = oracle.attn_rows(q, np.arange(S), k, v, [(0, S)], True, scale=0.5)
    c = 0.5 * (q[:, 0, :].astype(np.float64) @ k[0, 0].astype(np.float64))
    np.testing.assert_allclose(lse[:, 0], c + np.log(np.arange(1, S + 1)), atol=1e-13)
    want = np.cumsum(v.astype(np.float64), axis=0) / np.arange(1, S + 1)[:, None, None]
    np.testing.assert_allclose(o, want, atol=1e-13)


def test_single_key_returns_its_value_row():
    d = 16
    q, k, v = _rand((1, 2, d), 51), _rand((1, 2, d), 52), _rand((1, 2, d), 53)
    o, lse = oracle.attn_rows(q, [0], k, v, [(0, 1)], True)
    np.testing.assert_allclose(o, v.astype(np.float64), atol=1e-15)
    want = (q.astype(np.float64) * k.astype(np.float64)).sum(-1) / math.sqrt(d)
    np.testing.assert_allclose(lse, want, atol=1e-14)


def test_dominant_key_wins():
    S, d = 12, 4
    q = np.zeros((1, 1, d), np.float32); q[0, 0, 0] = 1.0
    k = np.zeros((S, 1, d), np.float32); k[7, 0, 0] = 60.0
    v = _rand((S, 1, d), 61)
    o, lse = oracle.attn_rows(q, [S - 1], k, v, [(0, S)], True, scale=1.0)
    np.testing.assert_allclose(o[0, 0], v[7, 0].astype(np.float64), atol=1e-12)
    assert abs(lse[0, 0] - 60.0) < 1e-12


def test_hand_worked_two_key_row():
    """tests/golden/two_key_softmax.txt: probabilities 1/3 and 2/3."""
    vals = [float(x) for line in open(os.path.join(GOLDEN, "two_key_softmax.txt"))
            if line.strip() and not line.startswith("#") for x in line.split()]
    p0, p1, lse_w, o0, o1 = vals
    d = 4
    q = np.zeros((1, 1, d), np.float32); q[0, 0, 0] = 1.0
    k = np.zeros((2, 1, d), np.float32); k[1, 0, 0] = np.float32(math.log(2.0))
    v = np.zeros((2, 1, d), np.float32); v[0, 0, 0] = 3.0; v[1, 0, 1] = 3.0
    o, lse = oracle.attn_rows(q, [1], k, v, [(0, 2)], True, scale=1.0)
    assert abs(o[0, 0, 0] - o0) < 1e-7 and abs(o[0, 0, 1] - o1) < 1e-7  # ln2 rounded to fp32
    assert abs(o[0, 0, 0] / 3.0 - p0) < 1e-7 and abs(o[0, 0, 1] / 3.0 - p1) < 1e-7
    assert abs(lse[0, 0] - lse_w) < 1e-7
    # the causal limit is inclusive (Eq. 4 sums up to the row's own token): row 0 sees key 0 only
    o, lse = oracle.attn_rows(q, [0], k, v, [(0, 2)], True, scale=1.0)
    assert o[0, 0, 0] == 3.0 and o[0, 0, 1] == 0.0 and lse[0, 0] == 0.0


def test_constant_score_shift_moves_lse_only():
    S, d = 33, 8
    q, k, v = _rand((1, 1, d), 71), _rand((S, 1, d), 72), _rand((S, 1, d), 73)
    q[:] = np.round(q * 4) / 4            # keep the shifted keys exact in fp32
    k[:] = np.round(k * 4) / 4
    u = np.zeros(d, np.float32); u[0] = 2.0
    shift = float(q[0, 0, 0]) * 2.0 * 0.25
    o1, l1 = oracle.attn_rows(q, [S - 1], k, v, [(0, S)], True, scale=0.25)
    o2, l2 = oracle.attn_rows(q, [S - 1], k + u, v, [(0, S)], True, scale=0.25)
    np.testing.assert_allclose(o1, o2, atol=1e-13)
    np.testing.assert_allclose(l2 - l1, shift, atol=1e-12)


def test_scale_default_is_inverse_sqrt_d():
    S, d = 9, 16
    q, k, v = _rand((S, 1, d), 81), _rand((S, 1, d), 82), _rand((S, 1, d), 83)
    a = oracle.attn_rows(q, np.arange(S), k, v, [(0, S)], True)
    b = oracle.attn_rows(q, np.arange(S), k, v, [(0, S)], True, scale=0.25)
    np.testing.assert_array_equal(a[0], b[0])
    np.testing.assert_array_equal(a[1], b[1])


def test_gqa_equals_mha_with_repeated_kv_heads():
    S, hq, hkv, d = 40, 6, 2, 8
    q, k, v = _rand((S, hq, d), 91), _rand((S, hkv, d), 92), _rand((S, hkv, d), 93)
    a = oracle.attn_rows(q, np.arange(S), k, v, [(0, S)], True)
    kr, vr = np.repeat(k, 3, axis=1), np.repeat(v, 3, axis=1)
    b = oracle.attn_rows(q, np.arange(S), kr, vr, [(0, S)], True)
    np.testing.assert_array_equal(a[0], b[0])
    np.testing.assert_array_equal(a[1], b[1])


# ------------------------------------------------------------------ merge
def test_merge_identity_commutative_associative():
    n, h, d = 17, 3, 5
    g = np.random.Generator(np.random.Philox(key=101))
    parts = [(g.standard_normal((n, h, d)), g.standard_normal((n, h)) * 3) for _ in range(3)]
    (oa, la), (ob, lb), (oc, lc) = parts
    zero = (np.zeros((n, h, d)), np.full((n, h), -np.inf))
    o, l = oracle.merge(oa, la, *zero)
    np.testing.assert_array_equal(o, oa); np.testing.assert_array_equal(l, la)
    o, l = oracle.merge(*zero, oa, la)
    np.testing.assert_array_equal(o, oa); np.testing.assert_array_equal(l, la)
    o, l = oracle.merge(*zero, *zero)
    assert (o == 0).all() and np.isneginf(l).all()
    ab, ba = oracle.merge(oa, la, ob, lb), oracle.merge(ob, lb, oa, la)
    np.testing.assert_allclose(ab[0], ba[0], atol=1e-15); np.testing.assert_allclose(ab[1], ba[1], atol=1e-15)
    left = oracle.merge(*ab, oc, lc)
    right = oracle.merge(oa, la, *oracle.merge(ob, lb, oc, lc))
    np.testing.assert_allclose(left[0], right[0], atol=1e-13)
    np.testing.assert_allclose(left[1], right[1], atol=1e-13)


def test_merge_closed_form_weights():
    """LSE_a = ln 1, LSE_b = ln 3 -> weights 1/4 and 3/4, LSE = ln 4 (plain arithmetic)."""
    oa = np.full((1, 1, 2), 8.0); ob = np.full((1, 1, 2), 4.0)
    o, l = oracle.merge(oa, np.array([[0.0]]), ob, np.array([[math.log(3.0)]]))
    np.testing.assert_allclose(o, 5.0, atol=1e-14)
    np.testing.assert_allclose(l, math.log(4.0), atol=1e-14)


def test_merge_of_disjoint_key_sets_is_attention_over_the_union():
    S, hq, hkv, d = 90, 4, 2, 16
    q, k, v = _rand((S, hq, d), 111), _rand((S, hkv, d), 112), _rand((S, hkv, d), 113)
    pos = np.arange(S)
    a = oracle.attn_rows(q, pos, k, v, [(0, 30), (70, 90)], True)
    b = oracle.attn_rows(q, pos, k, v, [(30, 70)], True)
    full = oracle.attn_rows(q, pos, k, v, [(0, S)], True)
    m = oracle.merge(*a, *b)
    np.testing.assert_allclose(m[0], full[0], atol=1e-13)
    np.testing.assert_allclose(m[1], full[1], atol=1e-13)
    # and against the library routine, so the chain attention -> merge is pinned end to end
    tq, tk, tv = (torch.from_numpy(x).double() for x in (q, k, v))
    tk, tv = tk.repeat_interleave(2, 1), tv.repeat_interleave(2, 1)
    ref = torch.nn.functional.scaled_dot_product_attention(
        tq.permute(1, 0, 2)[None], tk.permute(1, 0, 2)[None], tv.permute(1, 0, 2)[None], is_causal=True)
    np.testing.assert_allclose(m[0], ref[0].permute(1, 0, 2).numpy(), atol=1e-12)


def test_merge_n_equals_folded_pairwise_merges_and_attention_over_the_union():
    S, hq, hkv, d = 120, 4, 2, 16
    q, k, v = _rand((S, hq, d), 171), _rand((S, hkv, d), 172), _rand((S, hkv, d), 173)
    pos = np.arange(S)
    sets = [[(0, 10)], [(10, 50), (100, 120)], [(50, 51)], [(51, 100)], [(60, 60)]]   # last one empty
    parts = [oracle.attn_rows(q, pos, k, v, ivs, True) for ivs in sets]
    got = oracle.merge_n([p[0] for p in parts], [p[1] for p in parts])
    acc = parts[0]
    for part in parts[1:]:
        acc = oracle.merge(*acc, *part)
    np.testing.assert_allclose(got[0], acc[0], atol=1e-13)
    np.testing.assert_allclose(got[1], acc[1], atol=1e-13)
    full = oracle.attn_rows(q, pos, k, v, [(0, S)], True)
    np.testing.assert_allclose(got[0], full[0], atol=1e-12)
    np.testing.assert_allclose(got[1], full[1], atol=1e-12)
    tq = torch.from_numpy(q).double().permute(1, 0, 2)[None]
    tk = torch.from_numpy(k).double().repeat_interleave(2, 1).permute(1, 0, 2)[None]
    tv = torch.from_numpy(v).double().repeat_interleave(2, 1).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    np.testing.assert_allclose(got[0], ref[0].permute(1, 0, 2).numpy(), atol=1e-12)


def test_merge_n_closed_form_and_empty_rows():
    """LSE = ln 1, ln 2, ln 5 -> weights 1/8, 2/8, 5/8, LSE = ln 8 (plain arithmetic); garbage behind
    an empty part is ignored; all-empty rows give (0, -inf)."""
    o = [np.full((2, 1, 2), 8.0), np.full((2, 1, 2), 16.0), np.full((2, 1, 2), 1.6), np.full((2, 1, 2), np.nan)]
    l = [np.array([[0.0], [-np.inf]]), np.array([[math.log(2.0)], [-np.inf]]),
         np.array([[math.log(5.0)], [-np.inf]]), np.array([[-np.inf], [-np.inf]])]
    got_o, got_l = oracle.merge_n(o, l)
    np.testing.assert_allclose(got_o[0], 1.0 + 4.0 + 1.0, atol=1e-14)
    np.testing.assert_allclose(got_l[0], math.log(8.0), atol=1e-14)
    assert (got_o[1] == 0).all() and np.isneginf(got_l[1]).all()


# ------------------------------------------------------------------ the call-level oracle
@pytest.mark.parametrize("S,P,align", [(1024, 4, 128), (700, 3, 64), (130, 2, 128), (257, 8, 16)])
def test_partitions_merged_equal_monolithic(S, P, align):
    hq, hkv, d = 2, 1, 16
    q, k, v = _rand((S, hq, d), 121), _rand((S, hkv, d), 122), _rand((S, hkv, d), 123)
    full = oracle.prefill_attn(q, k, v, seq_len=S)
    acc = None
    for p in reversed(range(P)):     # any order
        part = oracle.prefill_attn(q, k, v, seq_len=S, part_id=p, num_parts=P, part_align=align)
        acc = part if acc is None else oracle.merge(*acc, *part)
    np.testing.assert_allclose(acc[0], full[0], atol=1e-12)
    np.testing.assert_allclose(acc[1], full[1], atol=1e-12)


def test_chunked_resumed_prefill_equals_monolithic():
    """A chunk started later with the stored K/V prefix continues to the same rows (Section 5.1)."""
    S, C = 300, 64
    q, k, v = _rand((S, 2, 8), 131), _rand((S, 2, 8), 132), _rand((S, 2, 8), 133)
    full = oracle.prefill_attn(q, k, v, seq_len=S)
    for c0 in range(0, S, C):
        n = min(C, S - c0)
        o, l = oracle.prefill_attn(q, k, v, seq_len=S, chunk_start=c0, chunk_len=n, kv_len=c0 + n)
        np.testing.assert_array_equal(o, full[0][c0:c0 + n])
        np.testing.assert_array_equal(l, full[1][c0:c0 + n])


def test_sampled_rows_equal_full_rows():
    S = 200
    q, k, v = _rand((S, 2, 8), 141), _rand((S, 1, 8), 142), _rand((S, 1, 8), 143)
    full = oracle.prefill_attn(q, k, v, seq_len=S, part_id=1, num_parts=2, part_align=8)
    rows = [0, 7, 8, 99, 100, 199]
    o, l = oracle.prefill_attn(q, k, v, seq_len=S, part_id=1, num_parts=2, part_align=8, rows=rows)
    np.testing.assert_array_equal(o, full[0][rows])
    np.testing.assert_array_equal(l, full[1][rows])


def test_varlen_batch_equals_each_request_alone():
    lens = [5, 0, 33, 1, 64]
    cu = np.concatenate([[0], np.cumsum(lens)])
    T = int(cu[-1])
    q, k, v = _rand((T, 4, 8), 151), _rand((T, 2, 8), 152), _rand((T, 2, 8), 153)
    o, l = oracle.varlen_attn(q, k, v, cu)
    for r, n in enumerate(lens):
        if n == 0:
            continue
        a, b = cu[r], cu[r + 1]
        tq = torch.from_numpy(q[a:b]).double().permute(1, 0, 2)[None]
        tk = torch.from_numpy(k[a:b]).double().repeat_interleave(2, 1).permute(1, 0, 2)[None]
        tv = torch.from_numpy(v[a:b]).double().repeat_interleave(2, 1).permute(1, 0, 2)[None]
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
        np.testing.assert_allclose(o[a:b], ref[0].permute(1, 0, 2).numpy(), atol=1e-12)
    assert np.isfinite(l).all()


def test_bf16_inputs_widen_exactly():
    S = 40
    q, k, v = (torch.from_numpy(_rand((S, 2, 8), s)).to(torch.bfloat16) for s in (161, 162, 163))
    a = oracle.attn_rows(q, np.arange(S), k, v, [(0, S)], True)
    b = oracle.attn_rows(q.float().numpy(), np.arange(S), k.float().numpy(), v.float().numpy(), [(0, S)], True)
    np.testing.assert_array_equal(a[0], b[0])


# ------------------------------------------------------------------ dense steps
def test_linear_matches_loops_identity_and_per_head_stacking():
    """Eq. 2 / Eq. 5 as y = x w^T: explicit loops on a tiny case, identity weights, and stacking the
    per-head W_Q, W_K, W_V row-wise gives the per-head products side by side."""
    x, w = _rand((5, 6), 201), _rand((4, 6), 202)
    y = oracle.linear(x, w)
    for i in range(5):
        for j in range(4):
            assert abs(y[i, j] - sum(float(x[i, c]) * float(w[j, c]) for c in range(6))) < 1e-12
    np.testing.assert_array_equal(oracle.linear(x, np.eye(6, dtype=np.float32)), x.astype(np.float64))
    wq, wk = _rand((3, 6), 203), _rand((2, 6), 204)
    both = oracle.linear(x, np.concatenate([wq, wk]))
    np.testing.assert_array_equal(both[:, :3], oracle.linear(x, wq))
    np.testing.assert_array_equal(both[:, 3:], oracle.linear(x, wk))


# --------------------------------------------------------------------------- rotary position encoding
def test_rope_matches_the_hand_worked_rotations():
    path = os.path.join(os.path.dirname(__file__), "golden", "rope_worked.txt")
    n = 0
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        head, vec, want = (part.split() for part in line.split("|"))
        d, theta, pos = int(head[0]), float(head[1]), int(head[2])
        got = oracle.rope(np.array([[float(x) for x in vec]]), [pos], theta, d, head_dim=d)
        np.testing.assert_allclose(got[0], [float(x) for x in want], rtol=0, atol=1e-14)
        n += 1
    assert n == 3


def test_rope_is_a_rotation_that_depends_on_relative_position_only():
    g = np.random.Generator(np.random.Philox(key=77))
    d, theta = 128, 500000.0
    qv, kv = g.standard_normal((1, 2 * d)), g.standard_normal((1, 2 * d))
    # position 0 changes nothing
    np.testing.assert_array_equal(oracle.rope(qv, [0], theta, 2 * d, d), qv)
    # every (i, i + d/2) pair keeps its length
    r = oracle.rope(qv, [12345], theta, 2 * d, d)
    for h0 in (0, d):
        before = qv[0, h0:h0 + d // 2] ** 2 + qv[0, h0 + d // 2:h0 + d] ** 2
        after = r[0, h0:h0 + d // 2] ** 2 + r[0, h0 + d // 2:h0 + d] ** 2
        np.testing.assert_allclose(after, before, rtol=1e-12)
    # q.k after the encoding depends on the distance of the two positions only (per head)
    for m, n in ((700, 300), (40000, 39600), (5, 405)):
        a = oracle.rope(qv, [m], theta, 2 * d, d)[0, :d] @ oracle.rope(kv, [n], theta, 2 * d, d)[0, :d]
        b = oracle.rope(qv, [m - n + 1000], theta, 2 * d, d)[0, :d] @ oracle.rope(kv, [1000], theta, 2 * d, d)[0, :d]
        np.testing.assert_allclose(a, b, rtol=0, atol=1e-9)
    # turning by a and then by b is turning by a + b
    twice = oracle.rope(oracle.rope(qv, [17], theta, 2 * d, d), [25], theta, 2 * d, d)
    np.testing.assert_allclose(twice, oracle.rope(qv, [42], theta, 2 * d, d), rtol=0, atol=1e-12)
    # the slowest pair of a head turns by position / theta**((d-2)/d): a quarter turn there swaps the pair
    pos = (np.pi / 2) * theta ** ((d - 2) / d)
    e = np.zeros((1, d)); e[0, d // 2 - 1] = 1.0
    out = oracle.rope(e, [pos], theta, d, d)
    np.testing.assert_allclose([out[0, d // 2 - 1], out[0, d - 1]], [0.0, 1.0], rtol=0, atol=1e-9)


def test_rope_leaves_the_value_columns_alone_and_shares_angles_between_heads():
    g = np.random.Generator(np.random.Philox(key=78))
    d = 128
    y = g.standard_normal((5, 4 * d))
    pos = [0, 1, 2, 1000, 77]
    out = oracle.rope(y, pos, 10000.0, 3 * d, d)
    np.testing.assert_array_equal(out[:, 3 * d:], y[:, 3 * d:])
    assert not np.allclose(out[1:, :3 * d], y[1:, :3 * d])
    # the same vector in two heads comes out the same
    y2 = np.concatenate([y[:, :d], y[:, :d]], axis=1)
    o2 = oracle.rope(y2, pos, 10000.0, 2 * d, d)
    np.testing.assert_array_equal(o2[:, :d], o2[:, d:])
    # rows are independent: a row's result depends on its own position only
    np.testing.assert_array_equal(oracle.rope(y[3:4], [1000], 10000.0, 3 * d, d), out[3:4])
    # linear_rope is the encoding of the projection
    x, w = g.standard_normal((5, 16)).astype(np.float32), g.standard_normal((4 * d, 16)).astype(np.float32)
    np.testing.assert_array_equal(oracle.linear_rope(x, w, pos, 10000.0, 3 * d, d), oracle.rope(oracle.linear(x, w), pos, 10000.0, 3 * d, d))

