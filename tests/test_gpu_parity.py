"""GPU parity: the CUDA path (through the C ABI) against the fp64 oracle, element by element,
at sizes that span several tiles and ragged tails, plus the degenerate cases."""
import numpy as np
import pytest
import torch

import oracle
from helpers import TOL, compare
from paper_2409_15104_b200 import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _qkv(seed, T, hq, hkv, dtype):
    q, k, v = workloads.qkv(seed, T, hq, hkv, 128, dtype)
    return q, k, v


def _gpu(*ts):
    return [t.to(DEV) for t in ts]


# ------------------------------------------------------------------ merge kernel
@pytest.mark.parametrize("rows,hq", [(1, 1), (33, 3), (1000, 8), (4096, 32), (77, 5)])
@pytest.mark.parametrize("mode", ["f32", "bf16", "inplace"])
def test_merge_matches_oracle(pec, rows, hq, mode):
    g = torch.Generator().manual_seed(rows * 131 + hq)
    oa, ob = torch.randn(rows, hq, 128, generator=g), torch.randn(rows, hq, 128, generator=g)
    la, lb = torch.randn(rows, hq, generator=g) * 4, torch.randn(rows, hq, generator=g) * 4
    # empty sides: a only, b only, both
    la[0::7] = float("-inf"); oa[0::7] = 0
    lb[3::5] = float("-inf"); ob[3::5] = 0
    want_o, want_l = oracle.merge(oa.numpy(), la.numpy(), ob.numpy(), lb.numpy())
    doa, dla, dob, dlb = _gpu(oa, la, ob, lb)
    if mode == "inplace":
        o, l = pec.pec_attn_merge(doa, dla, dob, dlb, inplace=True)
        assert o.data_ptr() == doa.data_ptr()
    else:
        o, l = pec.pec_attn_merge(doa, dla, dob, dlb, out_dtype=torch.float32 if mode == "f32" else torch.bfloat16)
    tol_o = 2e-2 if mode == "bf16" else 1e-5
    compare(o, l, want_o, want_l, tol_o, 1e-5, f"merge {mode}")


def test_merge_ignores_garbage_behind_an_empty_side(pec):
    rows, hq = 64, 4
    oa = torch.randn(rows, hq, 128); la = torch.randn(rows, hq)
    ob = torch.full((rows, hq, 128), float("nan")); lb = torch.full((rows, hq), float("-inf"))
    o, l = pec.pec_attn_merge(*_gpu(oa, la, ob, lb))
    assert torch.equal(o.cpu(), oa) and torch.equal(l.cpu(), la)


@pytest.mark.parametrize("n", [2, 3, 8, 16])
@pytest.mark.parametrize("mode", ["f32", "bf16", "inplace"])
def test_merge_n_matches_oracle(pec, n, mode):
    rows, hq = 517, 3
    g = torch.Generator().manual_seed(n * 17 + len(mode))
    os_ = [torch.randn(rows, hq, 128, generator=g) for _ in range(n)]
    ls_ = [torch.randn(rows, hq, generator=g) * 4 for _ in range(n)]
    for i in range(n):                                  # empty rows, different per part; rows 0..4 empty everywhere
        ls_[i][i::n + 1] = float("-inf"); os_[i][i::n + 1] = float("nan")
        ls_[i][:5] = float("-inf")
    want = oracle.merge_n([o.numpy() for o in os_], [l.numpy() for l in ls_])
    do, dl = [o.to(DEV) for o in os_], [l.to(DEV) for l in ls_]
    if mode == "inplace":
        o, l = pec.pec_attn_merge_n(do, dl, inplace=True)
        assert o.data_ptr() == do[0].data_ptr()
    else:
        o, l = pec.pec_attn_merge_n(do, dl, out_dtype=torch.float32 if mode == "f32" else torch.bfloat16)
    compare(o, l, *want, 2e-2 if mode == "bf16" else 1e-5, 1e-5, f"merge_n n={n} {mode}")


# ------------------------------------------------------------------ attention, single request
SHAPES = [  # (S, Hq, Hkv)
    (1, 1, 1), (2, 2, 1), (63, 2, 2), (64, 4, 2), (65, 2, 1), (127, 4, 4), (128, 8, 2), (129, 2, 2),
    (255, 4, 1), (257, 2, 2), (384, 8, 8), (1000, 4, 2),
]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("S,hq,hkv", SHAPES)
def test_full_causal_prefill(pec, dtype, S, hq, hkv):
    q, k, v = _qkv(1000 + S, S, hq, hkv, dtype)
    want = oracle.prefill_attn(q, k, v, seq_len=S)
    o, lse = pec.pec_prefill_attn(*_gpu(q, k, v))
    pec.check_status()
    assert o.dtype == dtype
    compare(o, lse, *want, *TOL[dtype], f"causal S={S} {dtype}")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_non_causal(pec, dtype):
    S = 300
    q, k, v = _qkv(2000, S, 4, 2, dtype)
    want = oracle.prefill_attn(q, k, v, seq_len=S, causal=False)
    o, lse = pec.pec_prefill_attn(*_gpu(q, k, v), causal=False)
    pec.check_status()
    compare(o, lse, *want, *TOL[dtype], "non-causal")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("S,P,align", [(1024, 4, 128), (700, 3, 64), (515, 2, 1), (130, 4, 128), (2048, 8, 128)])
def test_partition_partials_and_their_merge(pec, dtype, S, P, align):
    q, k, v = _qkv(3000 + S, S, 4, 2, dtype)
    dq, dk, dv = _gpu(q, k, v)
    acc = None
    for p in range(P):
        want = oracle.prefill_attn(q, k, v, seq_len=S, part_id=p, num_parts=P, part_align=align)
        o, lse = pec.pec_prefill_attn(dq, dk, dv, part_id=p, num_parts=P, part_align=align)
        pec.check_status()
        assert o.dtype == torch.float32
        compare(o, lse, *want, *TOL[dtype], f"partition {p}/{P} S={S}")
        acc = (o, lse) if acc is None else pec.pec_attn_merge(*acc, o, lse, inplace=True)
    full = oracle.prefill_attn(q, k, v, seq_len=S)
    compare(acc[0], acc[1], *full, *TOL[dtype], f"merged {P} partitions S={S}")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("S,C", [(1000, 256), (777, 100), (512, 128)])
def test_chunked_prefill_resumes_from_the_kv_prefix(pec, dtype, S, C):
    q, k, v = _qkv(4000 + S, S, 4, 1, dtype)
    dq, dk, dv = _gpu(q, k, v)
    want = oracle.prefill_attn(q, k, v, seq_len=S)
    o = torch.full((S, 4, 128), float("nan"), dtype=dtype, device=DEV)
    lse = torch.full((S, 4), float("nan"), dtype=torch.float32, device=DEV)
    for c0 in range(0, S, C):
        n = min(C, S - c0)
        # K/V beyond the prefix are poisoned: a resumed chunk must not read them
        kk, vv = dk.clone(), dv.clone()
        kk[c0 + n:] = float("nan"); vv[c0 + n:] = float("nan")
        pec.pec_prefill_attn(dq, kk, vv, seq_len=S, chunk_start=c0, chunk_len=n, kv_len=c0 + n,
                             o=o[c0:c0 + n], lse=lse[c0:c0 + n])
    pec.check_status()
    compare(o, lse, *want, *TOL[dtype], f"chunked S={S} C={C}")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_chunk_of_one_partition(pec, dtype):
    """A middle chunk against one zigzag partition cut by the K/V prefix."""
    S, P, c0, n = 1024, 4, 384, 200
    q, k, v = _qkv(5000, S, 2, 2, dtype)
    for p in range(P):
        want = oracle.prefill_attn(q, k, v, seq_len=S, chunk_start=c0, chunk_len=n, kv_len=c0 + n,
                                   part_id=p, num_parts=P)
        o, lse = pec.pec_prefill_attn(*_gpu(q, k, v), seq_len=S, chunk_start=c0, chunk_len=n, kv_len=c0 + n,
                                      part_id=p, num_parts=P)
        pec.check_status()
        compare(o, lse, *want, *TOL[dtype], f"chunk x partition {p}")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_strided_inputs_and_custom_scale(pec, dtype):
    """Q/K/V as slices of one fused [T, Hq+2Hkv, 128] projection output."""
    S, hq, hkv = 200, 4, 2
    fused = workloads.normal_tensor(6000, 1, (S, hq + 2 * hkv, 128), dtype)
    q, k, v = fused[:, :hq], fused[:, hq:hq + hkv], fused[:, hq + hkv:]
    want = oracle.prefill_attn(q, k, v, seq_len=S, scale=0.05)
    d = fused.to(DEV)
    o, lse = pec.pec_prefill_attn(d[:, :hq], d[:, hq:hq + hkv], d[:, hq + hkv:], softmax_scale=0.05)
    pec.check_status()
    compare(o, lse, *want, *TOL[dtype], "strided")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("shape", ["ramp", "spike", "falling"])
def test_row_maximum_that_moves(pec, dtype, shape):
    """Scores whose row maximum grows by far more than the lazy-rescale threshold (2^8) from one 64-key
    half to the next ("ramp"), jumps once in the middle of the key range ("spike"), or only falls
    ("falling": the accumulator is never rescaled).  Keys are multiples of one direction u, queries are u,
    so score(key j) = c_j |u|^2 with c_j chosen per shape; V stays random."""
    S, hq, hkv = 700, 2, 1
    q, k, v = _qkv(7100, S, hq, hkv, dtype)
    u = workloads.normal_tensor(7101, 1, (128,), torch.float32)
    u = u / u.norm() * (128 ** 0.25)                     # |u|^2 * scale = 1
    j = torch.arange(S, dtype=torch.float32)
    c = {"ramp": j * 0.2, "spike": torch.where(j == 333, torch.tensor(60.0), torch.tensor(0.0)) + 0.01 * torch.sin(j),
         "falling": (S - j) * 0.2}[shape]
    k = (c[:, None, None] * u[None, None, :]).expand(S, hkv, 128).to(dtype).contiguous()
    q = (u[None, None, :] * torch.ones(S, hq, 1)).to(dtype).contiguous()
    want = oracle.prefill_attn(q, k, v, seq_len=S)
    o, lse = pec.pec_prefill_attn(*_gpu(q, k, v))
    pec.check_status()
    compare(o, lse, *want, *TOL[dtype], f"moving maximum {shape} {dtype}")


# ------------------------------------------------------------------ packed batches
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("lens", [[5], [128, 128], [1, 300, 0, 77, 129, 64], [200, 1, 1, 511],
                                  [(i * 37) % 200 for i in range(70)]],      # more requests than one warp-wide search step
                         ids=["one", "two_tiles", "with_empty", "ragged", "seventy"])
def test_varlen_batch(pec, dtype, lens):
    cu = workloads.cu_seqlens(lens)
    T = cu[-1]
    q, k, v = _qkv(7000 + T, T, 4, 2, dtype)
    want = oracle.varlen_attn(q, k, v, cu)
    dcu = torch.tensor(cu, dtype=torch.int32, device=DEV)
    o, lse = pec.pec_prefill_attn(*_gpu(q, k, v), cu_seqlens=dcu)
    pec.check_status()
    compare(o, lse, *want, *TOL[dtype], f"varlen {lens}")


def test_bf16_partial_output_can_stay_fp32_or_round_to_bf16(pec):
    S = 256
    q, k, v = _qkv(8000, S, 2, 2, torch.bfloat16)
    want = oracle.prefill_attn(q, k, v, seq_len=S)
    o32, l32 = pec.pec_prefill_attn(*_gpu(q, k, v), out_dtype=torch.float32)
    o16, l16 = pec.pec_prefill_attn(*_gpu(q, k, v), out_dtype=torch.bfloat16)
    pec.check_status()
    compare(o32, l32, *want, 2e-2, 1e-3, "fp32 out")
    compare(o16, l16, *want, 2e-2, 1e-3, "bf16 out")
    assert torch.equal(l32, l16)
    assert torch.equal(o32.to(torch.bfloat16), o16)     # same accumulator, rounded once


def test_runs_are_bitwise_repeatable(pec):
    S = 640
    q, k, v = _gpu(*_qkv(9000, S, 4, 2, torch.bfloat16))
    a = pec.pec_prefill_attn(q, k, v)
    b = pec.pec_prefill_attn(q, k, v)
    pec.check_status()
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


def test_canaries_around_outputs_stay_untouched(pec):
    S, hq = 333, 2
    q, k, v = _gpu(*_qkv(9100, S, hq, 1, torch.bfloat16))
    pad = 64
    obuf = torch.full(((S + 2 * pad), hq, 128), 7.0, dtype=torch.bfloat16, device=DEV)
    lbuf = torch.full(((S + 2 * pad), hq), 7.0, dtype=torch.float32, device=DEV)
    pec.pec_prefill_attn(q, k, v, o=obuf[pad:pad + S], lse=lbuf[pad:pad + S])
    pec.check_status()
    assert (obuf[:pad] == 7).all() and (obuf[pad + S:] == 7).all()
    assert (lbuf[:pad] == 7).all() and (lbuf[pad + S:] == 7).all()


# ------------------------------------------------------------------ split-KV decode of a long request
@pytest.mark.parametrize("L,hq,hkv,lo,hi,splits", [
    (1, 4, 2, 0, 1, 0), (127, 8, 8, 0, 127, 0), (1000, 32, 8, 0, 1000, 0), (5000, 32, 8, 1234, 4999, 0),
    (4096, 64, 8, 0, 4096, 7), (3000, 16, 2, 0, 3000, 1), (777, 8, 2, 300, 300, 0), (20000, 32, 8, 0, 20000, 0),
])
@pytest.mark.parametrize("out", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_decode_split_kv(pec, L, hq, hkv, lo, hi, splits, out):
    _, k, v = _qkv(11000 + L, L, hq, hkv, torch.bfloat16)
    q = workloads.normal_tensor(11001 + L, 1, (1, hq, 128), torch.bfloat16)
    want = oracle.attn_rows(q, [L - 1], k, v, [(lo, hi)] if hi > lo else [], False)
    dq, dk, dv = _gpu(q[0], k, v)
    o, lse = pec.pec_decode_attn(dq, dk, dv, kv_lo=lo, kv_hi=hi, num_splits=splits, out_dtype=out)
    pec.check_status()
    compare(o[None], lse[None], *want, 2e-2, 1e-3, f"decode L={L} [{lo},{hi}) splits={splits}")


def test_decode_on_two_kv_halves_merges_to_the_whole(pec):
    """The colocation example: the long request's K/V split over two holders, partial outputs merged."""
    L, hq, hkv = 6000, 32, 8
    _, k, v = _qkv(12000, L, hq, hkv, torch.bfloat16)
    q = workloads.normal_tensor(12001, 1, (1, hq, 128), torch.bfloat16)
    dq, dk, dv = _gpu(q[0], k, v)
    a = pec.pec_decode_attn(dq, dk, dv, kv_lo=0, kv_hi=3100)
    b = pec.pec_decode_attn(dq, dk, dv, kv_lo=3100, kv_hi=L)
    o, lse = pec.pec_attn_merge(a[0][None], a[1][None], b[0][None], b[1][None], out_dtype=torch.bfloat16)
    pec.check_status()
    want = oracle.attn_rows(q, [L - 1], k, v, [(0, L)], False)
    compare(o, lse, *want, 2e-2, 1e-3, "decode halves merged")
    # decode of the last token equals the last row of a causal prefill of the same request
    qfull = torch.cat([workloads.normal_tensor(12002, 1, (L - 1, hq, 128), torch.bfloat16), q])
    po, pl = pec.pec_prefill_attn(qfull.to(DEV), dk, dv, chunk_start=L - 1, chunk_len=1, seq_len=L)
    pec.check_status()
    compare(po, pl, *want, 2e-2, 1e-3, "prefill last row")


# ------------------------------------------------------------------ the calls enqueue only: CUDA-graph capture
def test_partitioned_step_can_be_captured_and_replayed(pec):
    """No call allocates or synchronises, so a whole step (8 partials + n-way merge) captures into a CUDA
    graph; replays on new inputs match the eager result bit for bit."""
    from paper_2409_15104_b200.prefill import PartitionedPrefill
    S, hq, hkv, P = 2048, 8, 2, 4
    q, k, v = _gpu(*_qkv(13000, S, hq, hkv, torch.bfloat16))
    runner = PartitionedPrefill(S, hq, P, torch.bfloat16, DEV)
    o_eager, l_eager = (t.clone() for t in runner.run(q, k, v))       # also the warm-up outside capture
    pec.check_status()
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            runner.run(q, k, v, stream=stream)
    runner.out_o.zero_(); runner.out_l.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(runner.out_o, o_eager) and torch.equal(runner.out_l, l_eager)
    q2, k2, v2 = _gpu(*_qkv(13001, S, hq, hkv, torch.bfloat16))
    q.copy_(q2); k.copy_(k2); v.copy_(v2)                              # same buffers, new contents
    graph.replay()
    torch.cuda.synchronize()
    pec.check_status()
    want = oracle.prefill_attn(q2.cpu(), k2.cpu(), v2.cpu(), seq_len=S)
    compare(runner.out_o, runner.out_l, *want, 2e-2, 1e-3, "graph replay")


def test_decode_and_gemm_calls_capture_into_a_graph(pec):
    """A decode step (slice kernel + its dependent merge kernel), the QKV GEMM with rotary encoding and the Eq. 5 GEMM on
    unmerged partials, captured into one CUDA graph: the replay gives the eager calls' bits."""
    L, hq, hkv, T, d = 5000, 16, 2, 300, 256
    q, k, v = workloads.normal_tensor(14000, 1, (hq, 128), torch.bfloat16).to(DEV), *_gpu(*_qkv(14001, L, hq, hkv, torch.bfloat16)[1:])
    x = workloads.normal_tensor(14002, 1, (T, d), torch.bfloat16).to(DEV)
    w_qkv = (workloads.normal_tensor(14003, 2, ((hq + 2 * hkv) * 128, d), torch.float32) / d ** 0.5).to(torch.bfloat16).to(DEV)
    w_l = (workloads.normal_tensor(14004, 3, (d, hq * 128), torch.float32) / (hq * 128) ** 0.5).to(torch.bfloat16).to(DEV)
    tables = pec.pec_rope_table(500000.0, T, DEV)
    os_, ls_ = _random_partials(14005, T, hq, 2)
    os_, ls_ = [torch.nan_to_num(o).to(DEV) for o in os_], [l.to(DEV) for l in ls_]
    o = torch.empty((hq, 128), dtype=torch.float32, device=DEV); lse = torch.empty((hq,), dtype=torch.float32, device=DEV)
    a = pec.decode_args(q, k, v, o, lse, 0, L)
    ws = torch.empty(max(pec.pec_decode_workspace_size(a), 16), dtype=torch.uint8, device=DEV)
    y1 = torch.empty((T, (hq + 2 * hkv) * 128), dtype=torch.bfloat16, device=DEV)
    y2 = torch.empty((T, d), dtype=torch.bfloat16, device=DEV)

    def calls(stream=None):
        pec.pec_decode_attn(q, k, v, o=o, lse=lse, workspace=ws, stream=stream)
        pec.pec_linear_rope(x, w_qkv, tables, (hq + hkv) * 128, y=y1, stream=stream)
        pec.pec_linear_merged(os_, ls_, w_l, y=y2, stream=stream)

    calls()
    torch.cuda.synchronize()
    pec.check_status()
    eager = [t.clone() for t in (o, lse, y1, y2)]
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            calls(stream)
    for t in (o, lse, y1, y2):
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    pec.check_status()
    for got, want in zip((o, lse, y1, y2), eager):
        assert torch.equal(got, want)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_non_causal_partition_of_a_chunk(pec, dtype):
    S, P, c0, n = 900, 3, 256, 300
    q, k, v = _qkv(14000, S, 4, 2, dtype)
    for p in range(P):
        want = oracle.prefill_attn(q, k, v, seq_len=S, chunk_start=c0, chunk_len=n, kv_len=700, part_id=p,
                                   num_parts=P, part_align=32, causal=False)
        o, lse = pec.pec_prefill_attn(*_gpu(q, k, v), seq_len=S, chunk_start=c0, chunk_len=n, kv_len=700, part_id=p,
                                      num_parts=P, part_align=32, causal=False)
        pec.check_status()
        compare(o, lse, *want, *TOL[dtype], f"non-causal chunk x partition {p}")


# ------------------------------------------------------------------ dense steps either side of the attention
@pytest.mark.parametrize("M,N,K", [(1, 8, 8), (128, 256, 64), (130, 264, 72), (1000, 768, 512), (257, 6144, 4096),
                                   (4096, 128, 1024)])
def test_linear_matches_oracle(pec, M, N, K):
    x = workloads.normal_tensor(15000 + M, 1, (M, K), torch.bfloat16)
    w = (workloads.normal_tensor(15001 + N, 2, (N, K), torch.float32) / K ** 0.5).to(torch.bfloat16)
    want = oracle.linear(x, w)
    y = pec.pec_linear(x.to(DEV), w.to(DEV))
    pec.check_status()
    err = np.abs(y.float().cpu().double().numpy() - want).max()
    print(f"[parity] linear {M}x{N}x{K}: max|dy| = {err:.3e}")
    assert err <= 2e-2                                   # outputs ~ N(0,1); bf16 rounding of the result dominates


def test_attention_layer_steps_chain_through_strides(pec):
    """Eq. 2 -> Eq. 3 -> Eq. 5 on the GPU: fused QKV projection, attention reading q/k/v as strided slices of
    it, output projection; each step checked against the oracle applied to that step's actual inputs."""
    T, d, hq, hkv = 600, 512, 4, 2
    e = workloads.normal_tensor(16000, 1, (T, d), torch.bfloat16)
    w_qkv = (workloads.normal_tensor(16001, 2, ((hq + 2 * hkv) * 128, d), torch.float32) / d ** 0.5).to(torch.bfloat16)
    w_l = (workloads.normal_tensor(16002, 3, (d, hq * 128), torch.float32) / (hq * 128) ** 0.5).to(torch.bfloat16)
    qkv = pec.pec_linear(e.to(DEV), w_qkv.to(DEV))
    fused = qkv.view(T, hq + 2 * hkv, 128)
    q, k, v = fused[:, :hq], fused[:, hq:hq + hkv], fused[:, hq + hkv:]
    o, lse = pec.pec_prefill_attn(q, k, v)
    out = pec.pec_linear(o.view(T, hq * 128), w_l.to(DEV))
    pec.check_status()
    assert np.abs(qkv.float().cpu().double().numpy() - oracle.linear(e, w_qkv)).max() <= 2e-2
    want = oracle.prefill_attn(q.cpu(), k.cpu(), v.cpu(), seq_len=T)
    compare(o, lse, *want, 2e-2, 1e-3, "attention on projected q, k, v")
    assert np.abs(out.float().cpu().double().numpy() - oracle.linear(o.view(T, hq * 128).cpu(), w_l)).max() <= 2e-2


def test_rope_table_matches_fp64_cos_and_sin(pec):
    """The two-level table, combined the way the kernel combines it, against cos and sin of the angles in fp64."""
    theta, n_pos = 500000.0, 70001
    tables = pec.pec_rope_table(theta, n_pos, DEV)
    cos, sin = pec.rope_table_angles(tables)
    ang = np.arange(n_pos, dtype=np.float64)[:, None] * theta ** (-2.0 * np.arange(64, dtype=np.float64) / 128)[None, :]
    assert np.abs(cos.numpy() - np.cos(ang)).max() <= 3e-7
    assert np.abs(sin.numpy() - np.sin(ang)).max() <= 3e-7


@pytest.mark.parametrize("M,N,K,rot,pos0", [(1, 128, 8, 128, 0), (130, 384, 72, 256, 5), (257, 6144, 512, 5120, 65000),
                                            (600, 392, 64, 384, 499_000), (300, 256, 128, 0, 3)])
def test_linear_rope_matches_oracle(pec, M, N, K, rot, pos0):
    """Eq. 2 with the rotary encoding of the query and key heads in the GEMM's epilogue; rows are a chunk at pos0."""
    theta = 500000.0
    x = workloads.normal_tensor(18000 + M, 1, (M, K), torch.bfloat16)
    w = (workloads.normal_tensor(18001 + N, 2, (N, K), torch.float32) / K ** 0.5).to(torch.bfloat16)
    tables = pec.pec_rope_table(theta, pos0 + M, DEV)
    y = pec.pec_linear_rope(x.to(DEV), w.to(DEV), tables, rot, pos0=pos0)
    pec.check_status()
    want = oracle.linear_rope(x, w, np.arange(pos0, pos0 + M), theta, rot)
    err = np.abs(y.float().cpu().double().numpy() - want).max()
    print(f"[parity] linear_rope {M}x{N}x{K} rot={rot} pos0={pos0}: max|dy| = {err:.3e}")
    assert err <= 2e-2
    if rot == 0:                                          # nothing to turn: the plain GEMM's bits
        assert torch.equal(y, pec.pec_linear(x.to(DEV), w.to(DEV)))


def test_linear_rope_packed_positions_and_attention_on_the_encoded_heads(pec):
    """A packed batch: every row carries its position inside its own request; the encoded q and k then go through
    the attention as strided slices, and each step is compared with the oracle applied to that step's inputs."""
    lens, d, hq, hkv, theta = [300, 1, 515, 128], 256, 4, 2, 10000.0
    cu = workloads.cu_seqlens(lens)
    T = cu[-1]
    pos = np.concatenate([np.arange(n) for n in lens]).astype(np.int32)
    e = workloads.normal_tensor(18100, 1, (T, d), torch.bfloat16)
    w_qkv = (workloads.normal_tensor(18101, 2, ((hq + 2 * hkv) * 128, d), torch.float32) / d ** 0.5).to(torch.bfloat16)
    tables = pec.pec_rope_table(theta, max(lens), DEV)
    qkv = pec.pec_linear_rope(e.to(DEV), w_qkv.to(DEV), tables, (hq + hkv) * 128, positions=torch.from_numpy(pos).to(DEV))
    pec.check_status()
    want = oracle.linear_rope(e, w_qkv, pos, theta, (hq + hkv) * 128)
    assert np.abs(qkv.float().cpu().double().numpy() - want).max() <= 2e-2
    fused = qkv.view(T, hq + 2 * hkv, 128)
    q, k, v = fused[:, :hq], fused[:, hq:hq + hkv], fused[:, hq + hkv:]
    o, lse = pec.pec_prefill_attn(q, k, v, cu_seqlens=torch.tensor(cu, dtype=torch.int32, device=DEV))
    pec.check_status()
    compare(o, lse, *oracle.varlen_attn(q.cpu(), k.cpu(), v.cpu(), cu), 2e-2, 1e-3, "attention on rotary-encoded q, k")


def _random_partials(seed, rows, hq, n):
    """n fp32 partials with LSEs; about a fifth of the (row, head, part) entries empty (lse = -inf, o poisoned with NaN:
    an empty part must not be read), and a few rows empty in every part."""
    g = torch.Generator().manual_seed(seed)
    os_, ls_ = [], []
    dead_rows = torch.rand((rows, 1), generator=g) < 0.03
    for i in range(n):
        o = workloads.normal_tensor(seed + 10 * i, 1, (rows, hq, 128), torch.float32)
        l = workloads.normal_tensor(seed + 10 * i + 1, 2, (rows, hq), torch.float32) * 3.0
        empty = (torch.rand((rows, hq), generator=g) < 0.2) | dead_rows
        l[empty] = float("-inf")
        o[empty] = float("nan")
        os_.append(o)
        ls_.append(l)
    return os_, ls_


@pytest.mark.parametrize("rows,hq,N,n", [(1, 1, 8, 1), (100, 1, 72, 2), (256, 2, 512, 2), (300, 4, 520, 3), (700, 3, 1024, 4),
                                         (513, 2, 1288, 8), (2048, 32, 4096, 2)])
def test_linear_merged_matches_oracle(pec, rows, hq, N, n):
    """Eq. 5 on the merge of n partials (Section 2.2, Section 5.2): against merge_n -> linear of the oracle."""
    os_, ls_ = _random_partials(17000 + rows + n, rows, hq, n)
    K = hq * 128
    w = (workloads.normal_tensor(17001 + N, 3, (N, K), torch.float32) / K ** 0.5).to(torch.bfloat16)
    merged, _ = oracle.merge_n([torch.nan_to_num(o, nan=0.0).numpy() for o in os_], [l.numpy() for l in ls_])
    want = oracle.linear(torch.from_numpy(merged.reshape(rows, K)), w)
    y = pec.pec_linear_merged([o.to(DEV) for o in os_], [l.to(DEV) for l in ls_], w.to(DEV))
    pec.check_status()
    got = y.float().cpu().double().numpy()
    assert np.isfinite(got).all()
    err = np.abs(got - want).max()
    print(f"[parity] linear_merged rows={rows} Hq={hq} N={N} n={n}: max|dy| = {err:.3e}")
    assert err <= 2e-2                                   # bf16 rounding of the merged operand and of the result
    # the unfused route through the merge kernel and pec_linear rounds the same merged values the same way
    if n >= 2:
        o_m, _ = pec.pec_attn_merge_n([torch.nan_to_num(o, nan=0.0).to(DEV) for o in os_], [l.to(DEV) for l in ls_],
                                      out_dtype=torch.bfloat16)
        y2 = pec.pec_linear(o_m.view(rows, K), w.to(DEV))
        pec.check_status()
        assert (y2.float() - y.float()).abs().max().item() <= 2e-2


def test_linear_merged_on_partitioned_attention(pec):
    """Two key partitions' partial attention (the two GPUs' O_1, O_2 of Section 5.2) go into Eq. 5 unmerged."""
    S, hq, hkv, d = 1536, 4, 2, 384
    q, k, v = _qkv(workloads.BASE_SEED + 170, S, hq, hkv, torch.bfloat16)
    w_l = (workloads.normal_tensor(17100, 3, (d, hq * 128), torch.float32) / (hq * 128) ** 0.5).to(torch.bfloat16)
    parts = [pec.pec_prefill_attn(*_gpu(q, k, v), part_id=i, num_parts=2, part_align=64, out_dtype=torch.float32) for i in range(2)]
    y = pec.pec_linear_merged([o for o, _ in parts], [l for _, l in parts], w_l.to(DEV))
    pec.check_status()
    want_o, _ = oracle.prefill_attn(q, k, v, seq_len=S)
    want = oracle.linear(torch.from_numpy(np.asarray(want_o).reshape(S, hq * 128)), w_l)
    err = np.abs(y.float().cpu().double().numpy() - want).max()
    print(f"[parity] attention partials -> linear_merged: max|dy| = {err:.3e}")
    assert err <= 2e-2


# ------------------------------------------------------------------ ring-attention step form
@pytest.mark.parametrize("S,P,hq,hkv", [(2048, 4, 4, 2), (1500, 3, 2, 1), (700, 1, 2, 2), (300, 8, 2, 1)])
def test_ring_prefill_every_rank_and_step_equals_monolithic(pec, S, P, hq, hkv):
    from paper_2409_15104_b200 import prefill
    q, k, v = _qkv(workloads.BASE_SEED + 70 + P, S, hq, hkv, torch.bfloat16)
    o, lse, launches = prefill.ring_prefill(*_gpu(q, k, v), num_parts=P, part_align=64)
    pec.check_status()
    want_o, want_l = oracle.prefill_attn(q, k, v, seq_len=S)
    compare(o, lse, want_o, want_l, *TOL[torch.bfloat16], f"ring S={S} P={P}")
    assert launches == P * P                         # one launch per (rank, ring step), merges included
    # the plan's per-step work adds up to the causal total the launches computed
    assert sum(pec.pec_plan_ring(S, P, 64)["rank_total"]) == S * (S + 1) // 2


# ------------------------------------------------------------------ seeded random call shapes
def _random_call(seed):
    g = np.random.Generator(np.random.Philox(key=9000 + seed))
    S = int(g.integers(1, 1400))
    hkv = int(g.choice([1, 2, 4]))
    hq = hkv * int(g.choice([1, 2, 4]))
    P = int(g.choice([1, 1, 2, 3, 4, 8]))
    align = int(g.choice([1, 16, 64, 128]))
    causal = bool(g.integers(0, 4) > 0)
    c0 = int(g.integers(0, S))
    n = int(g.integers(1, S - c0 + 1))
    kv_len = int(g.integers(c0 + n, S + 1)) if causal else int(g.integers(1, S + 1))
    return dict(S=S, hq=hq, hkv=hkv, P=P, part=int(g.integers(0, P)), align=align, causal=causal, c0=c0, n=n, kv_len=kv_len)


@pytest.mark.parametrize("seed", range(24))
def test_random_chunk_partition_prefix_combinations(pec, seed):
    """Chunk start/length, K/V prefix, partition, alignment, GQA ratio and mask drawn from a seed: the two
    stages of a CTA then see different numbers of key tiles, none at all, or a single ragged one."""
    c = _random_call(seed)
    q, k, v = _qkv(9100 + seed, c["S"], c["hq"], c["hkv"], torch.bfloat16)
    want = oracle.prefill_attn(q, k, v, seq_len=c["S"], chunk_start=c["c0"], chunk_len=c["n"], kv_len=c["kv_len"],
                               part_id=c["part"], num_parts=c["P"], part_align=c["align"], causal=c["causal"])
    dq, dk, dv = _gpu(q, k, v)
    dk[c["kv_len"]:] = float("nan"); dv[c["kv_len"]:] = float("nan")     # nothing past the prefix may be read
    o, lse = pec.pec_prefill_attn(dq, dk, dv, seq_len=c["S"], chunk_start=c["c0"], chunk_len=c["n"], kv_len=c["kv_len"],
                                  part_id=c["part"], num_parts=c["P"], part_align=c["align"], causal=c["causal"],
                                  out_dtype=torch.float32)
    pec.check_status()
    compare(o, lse, *want, *TOL[torch.bfloat16], f"random call {c}")


def test_streamed_prefill_matches_one_step_at_a_time(pec):
    """Five consecutive host-to-host steps with different inputs through the three-stream pipeline: every
    result equals (bit for bit) what the same runner gives for that input alone."""
    from paper_2409_15104_b200.prefill import PartitionedPrefill, StreamedPrefill
    S, hq, hkv, P = 1536, 4, 2, 4
    runner = PartitionedPrefill(S, hq, P, torch.bfloat16, DEV)
    pipe = StreamedPrefill(runner, hkv, DEV)
    steps = []
    for i in range(5):
        q, k, v = (t.pin_memory() for t in _qkv(workloads.BASE_SEED + 300 + i, S, hq, hkv, torch.bfloat16))
        o_h = torch.empty((S, hq, 128), dtype=torch.bfloat16).pin_memory()
        l_h = torch.empty((S, hq), dtype=torch.float32).pin_memory()
        steps.append((q, k, v, o_h, l_h))
    for st in steps:
        pipe.submit(*st)
    pipe.drain()
    pec.check_status()
    for i, (q, k, v, o_h, l_h) in enumerate(steps):
        o, l = runner.run(*_gpu(q, k, v))
        torch.cuda.synchronize()
        assert torch.equal(o.cpu(), o_h) and torch.equal(l.cpu(), l_h), f"step {i}"
    want_o, want_l = oracle.prefill_attn(steps[-1][0], steps[-1][1], steps[-1][2], seq_len=S)
    compare(steps[-1][3], steps[-1][4], want_o, want_l, *TOL[torch.bfloat16], "streamed, last step")


# ------------------------------------------------------------------ incoming state: online softmax across launches
def _orders(P):
    return {"ascending": list(range(P)), "descending": list(range(P - 1, -1, -1)),
            "interleaved": list(range(1, P, 2)) + list(range(0, P, 2))}


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("S,P,align,order", [(1024, 4, 128, "ascending"), (700, 3, 64, "descending"), (515, 2, 1, "ascending"),
                                             (130, 4, 128, "descending"), (2048, 8, 128, "interleaved"), (1500, 5, 32, "interleaved")])
def test_chain_of_partition_launches_equals_monolithic(pec, dtype, S, P, align, order):
    """Each launch merges its partition's result into the state the previous launches left (in place), the
    last one writing the final output in the input dtype.  After every launch the state equals the oracle's
    merge of the partials so far; at the end it equals the monolithic result."""
    q, k, v = _qkv(17000 + S, S, 4, 2, dtype)
    dq, dk, dv = _gpu(q, k, v)
    seq = _orders(P)[order]
    st_o = torch.full((S, 4, 128), float("nan"), dtype=torch.float32, device=DEV)
    st_l = torch.full((S, 4), float("nan"), dtype=torch.float32, device=DEV)
    want = None
    for i, part in enumerate(seq[:-1]):
        own = oracle.prefill_attn(q, k, v, seq_len=S, part_id=part, num_parts=P, part_align=align)
        want = own if want is None else oracle.merge(*want, *own)
        pec.pec_prefill_attn(dq, dk, dv, part_id=part, num_parts=P, part_align=align, o=st_o, lse=st_l,
                             acc=None if i == 0 else (st_o, st_l))
        pec.check_status()
        compare(st_o, st_l, *want, *TOL[dtype], f"state after {i + 1} of {P} launches ({order})")
    o, lse = pec.pec_prefill_attn(dq, dk, dv, part_id=seq[-1], num_parts=P, part_align=align, acc=(st_o, st_l), out_dtype=dtype)
    pec.check_status()
    assert o.dtype == dtype and o.data_ptr() != st_o.data_ptr()
    compare(o, lse, *oracle.prefill_attn(q, k, v, seq_len=S), *TOL[dtype], f"chain of {P} launches ({order})")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_incoming_state_with_empty_rows_on_either_side(pec, dtype):
    """Rows empty in the state only, in the launch's own result only, in both, in neither; the incoming state's
    buffers are separate from the outputs here and must come back unchanged."""
    S, P = 1300, 4
    q, k, v = _qkv(17100, S, 2, 1, dtype)
    dq, dk, dv = _gpu(q, k, v)
    # state: partition 2 over a short prefix (rows below 2b are empty); own: partition 3 (rows below 3b are empty)
    a_o, a_l = pec.pec_prefill_attn(dq, dk, dv, part_id=2, num_parts=P, part_align=16, out_dtype=torch.float32)
    keep_o, keep_l = a_o.clone(), a_l.clone()
    want_a = oracle.prefill_attn(q, k, v, seq_len=S, part_id=2, num_parts=P, part_align=16)
    want_b = oracle.prefill_attn(q, k, v, seq_len=S, part_id=3, num_parts=P, part_align=16)
    assert np.isneginf(want_a[1]).any() and np.isneginf(want_b[1]).any()
    for out in (torch.float32, dtype):
        o, lse = pec.pec_prefill_attn(dq, dk, dv, part_id=3, num_parts=P, part_align=16, acc=(a_o, a_l), out_dtype=out)
        pec.check_status()
        compare(o, lse, *oracle.merge(*want_a, *want_b), *TOL[dtype], f"state + own, out {out}")
        assert torch.equal(a_o, keep_o) and torch.equal(a_l, keep_l)
    # the other way round: the state has keys where the launch has none
    b_o, b_l = pec.pec_prefill_attn(dq, dk, dv, part_id=3, num_parts=P, part_align=16, out_dtype=torch.float32)
    o, lse = pec.pec_prefill_attn(dq, dk, dv, part_id=0, num_parts=P, part_align=16, acc=(b_o, b_l), out_dtype=torch.float32)
    pec.check_status()
    compare(o, lse, *oracle.merge(*want_b, *oracle.prefill_attn(q, k, v, seq_len=S, part_id=0, num_parts=P, part_align=16)),
            *TOL[dtype], "own + state")


@pytest.mark.parametrize("seed", range(12))
def test_random_chunk_partition_prefix_combinations_with_incoming_state(pec, seed):
    """Two launches over different key partitions of a random chunk / prefix / alignment: the second takes the
    first one's result as its incoming state, in place on even seeds, into a separate bf16 output on odd ones."""
    c = _random_call(100 + seed)
    if c["P"] == 1:
        c["P"] = 3
    c["part"] = c["part"] % c["P"]
    other = (c["part"] + 1 + seed % (c["P"] - 1)) % c["P"]
    q, k, v = _qkv(9300 + seed, c["S"], c["hq"], c["hkv"], torch.bfloat16)
    kw = dict(seq_len=c["S"], chunk_start=c["c0"], chunk_len=c["n"], kv_len=c["kv_len"], num_parts=c["P"],
              part_align=c["align"], causal=c["causal"])
    want = oracle.merge(*oracle.prefill_attn(q, k, v, part_id=c["part"], **kw), *oracle.prefill_attn(q, k, v, part_id=other, **kw))
    dq, dk, dv = _gpu(q, k, v)
    dk[c["kv_len"]:] = float("nan"); dv[c["kv_len"]:] = float("nan")
    st_o, st_l = pec.pec_prefill_attn(dq, dk, dv, part_id=c["part"], out_dtype=torch.float32, **kw)
    if seed % 2 == 0:
        o, lse = pec.pec_prefill_attn(dq, dk, dv, part_id=other, o=st_o, lse=st_l, acc=(st_o, st_l), **kw)
    else:
        o, lse = pec.pec_prefill_attn(dq, dk, dv, part_id=other, acc=(st_o, st_l), out_dtype=torch.bfloat16, **kw)
    pec.check_status()
    compare(o, lse, *want, *TOL[torch.bfloat16], f"random call with state {c} + partition {other}")


# ------------------------------------------------------------------ a ring rank's rows in one launch
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("S,P,align,c0,n", [(1024, 4, 128, 0, 1024), (1500, 3, 64, 0, 1500), (900, 2, 1, 100, 700), (300, 8, 16, 0, 300)])
def test_query_partition_launch_touches_only_its_rows(pec, dtype, S, P, align, c0, n):
    q, k, v = _qkv(18000 + S, S, 4, 2, dtype)
    dq, dk, dv = _gpu(q, k, v)
    for r in range(P):
        rows = oracle.partition_rows(S, P, r, align, c0, n)
        for s in {(r - 1) % P, r, (r + 1) % P}:
            o = torch.full((n, 4, 128), 7.0, dtype=torch.float32, device=DEV)
            lse = torch.full((n, 4), 7.0, dtype=torch.float32, device=DEV)
            pec.pec_prefill_attn(dq, dk, dv, seq_len=S, chunk_start=c0, chunk_len=n, kv_len=S, part_id=s, num_parts=P,
                                 part_align=align, q_part_id=r, q_num_parts=P, o=o, lse=lse)
            pec.check_status()
            mine = torch.zeros(n, dtype=torch.bool)
            if rows:
                idx = torch.as_tensor(rows) - c0
                mine[idx] = True
                want = oracle.prefill_attn(q, k, v, seq_len=S, chunk_start=c0, chunk_len=n, kv_len=S, part_id=s, num_parts=P,
                                           part_align=align, rows=rows)
                compare(o[idx.to(DEV)], lse[idx.to(DEV)], *want, *TOL[dtype], f"rank {r} rows x keys of {s}")
            assert (o.cpu()[~mine] == 7).all() and (lse.cpu()[~mine] == 7).all(), "rows of other ranks were written"


# ------------------------------------------------------------------ packed batch through a work-list
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("lens", [[5], [1, 300, 0, 77, 129, 64], [700, 20, 1200, 256, 257], [(i * 37) % 200 for i in range(70)]],
                         ids=["one", "with_empty", "mixed", "seventy"])
def test_varlen_batch_through_a_worklist(pec, dtype, lens):
    from paper_2409_15104_b200 import prefill
    cu = workloads.cu_seqlens(lens)
    T = cu[-1]
    q, k, v = _qkv(19000 + T, T, 4, 2, dtype)
    dq, dk, dv = _gpu(q, k, v)
    dcu = torch.tensor(cu, dtype=torch.int32, device=DEV)
    wl = prefill.make_worklist(cu, dtype, DEV)
    assert wl.shape == (sum(-(-n // pec.pec_worklist_block_m(dtype)) for n in lens), 4)
    o, lse = prefill.varlen_prefill(dq, dk, dv, dcu, worklist=wl)
    o2, lse2 = prefill.varlen_prefill(dq, dk, dv, dcu)
    pec.check_status()
    compare(o, lse, *oracle.varlen_attn(q, k, v, cu), *TOL[dtype], f"varlen work-list {lens[:6]}")
    assert torch.equal(o, o2) and torch.equal(lse, lse2)          # same tiles, another order


# ------------------------------------------------------------------ the two ways a partitioned step combines its partitions
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("budget_parts", [2, 3, 16])
def test_partitioned_prefill_by_merge_passes_equals_the_chained_form(pec, dtype, budget_parts):
    """chain=False keeps partials and merges them n at a time (2: the running two-way merge; 3: several n-way
    groups; 16: one pass); chain=True merges in the attention epilogue.  Both against the oracle."""
    from paper_2409_15104_b200.prefill import PartitionedPrefill
    S, hq, hkv, P = 1536, 4, 2, 6
    q, k, v = _qkv(20000 + budget_parts, S, hq, hkv, dtype)
    dq, dk, dv = _gpu(q, k, v)
    want = oracle.prefill_attn(q, k, v, seq_len=S)
    per_partial = S * hq * (128 * 4 + 4)
    merged = PartitionedPrefill(S, hq, P, dtype, DEV, part_align=64, partial_budget_bytes=budget_parts * per_partial, chain=False)
    assert merged.max_live == min(budget_parts, P)
    o, lse = merged.run(dq, dk, dv)
    pec.check_status()
    compare(o, lse, *want, *TOL[dtype], f"merge passes, {merged.max_live} partials live")
    assert len(merged.merge_parts) == merged.merge_launches()
    chained = PartitionedPrefill(S, hq, P, dtype, DEV, part_align=64)
    o2, lse2 = chained.run(dq, dk, dv)
    pec.check_status()
    compare(o2, lse2, *want, *TOL[dtype], "chained")


def test_launches_that_overlap_their_predecessor_give_the_same_bits(pec):
    """overlap_previous lets a launch start on the SMs its predecessor has left; it must still see the complete
    incoming state.  A chain of short launches (many more CTAs than SMs, state merged in place) run both ways,
    several times over, gives identical bits; the chain equals the monolithic oracle result."""
    S, hq, hkv, P = 4096, 16, 4, 8
    q, k, v = _qkv(22000, S, hq, hkv, torch.bfloat16)
    dq, dk, dv = _gpu(q, k, v)

    def chain(overlap):
        st_o = torch.full((S, hq, 128), float("nan"), dtype=torch.float32, device=DEV)
        st_l = torch.full((S, hq), float("nan"), dtype=torch.float32, device=DEV)
        pec.pec_prefill_attn(dq, dk, dv, part_id=1, num_parts=P, o=st_o, lse=st_l)
        for part in range(2, P):
            pec.pec_prefill_attn(dq, dk, dv, part_id=part, num_parts=P, o=st_o, lse=st_l, acc=(st_o, st_l), overlap_previous=overlap)
        return pec.pec_prefill_attn(dq, dk, dv, part_id=0, num_parts=P, acc=(st_o, st_l), out_dtype=torch.bfloat16,
                                    overlap_previous=overlap)

    base = chain(False)
    pec.check_status()
    for _ in range(5):
        o, lse = chain(True)
        pec.check_status()
        assert torch.equal(o, base[0]) and torch.equal(lse, base[1])
    compare(o, lse, *oracle.prefill_attn(q, k, v, seq_len=S), *TOL[torch.bfloat16], "overlapping chain")


# ------------------------------------------------------------------ many random calls, the two kernels against each other
def test_many_random_calls_bf16_kernel_against_fp32_kernel(pec):
    """A cross-check beside the oracle comparisons above, not instead of them: 600 seeded calls (lengths to 9000, chunks,
    prefixes, key partitions, query partitions, incoming state, fused-QKV strides, score scales, moved maxima) through the
    tensor-core kernel and through the fp32 kernel (itself compared with the oracle in full elsewhere) on the same
    inputs; every element of O and LSE must agree and the same rows must be empty."""
    worst_o = worst_l = 0.0
    for seed in range(600):
        g = np.random.Generator(np.random.Philox(key=777000 + seed))
        S = int(g.integers(1, 9000)) if seed % 3 else int(g.integers(1, 700))
        hkv = int(g.choice([1, 2, 3]))
        hq = hkv * int(g.choice([1, 2, 4, 8]))
        P = int(g.choice([1, 1, 2, 3, 4, 8, 16]))
        align = int(g.choice([1, 16, 64, 128, 256]))
        causal = bool(g.integers(0, 5) > 0)
        c0 = int(g.integers(0, S)) if g.integers(0, 2) else 0
        n = int(g.integers(1, S - c0 + 1)) if g.integers(0, 2) else S - c0
        kv_len = int(g.integers(c0 + n, S + 1)) if causal else int(g.integers(1, S + 1))
        part = int(g.integers(0, P))
        qP = int(g.choice([0, 0, 2, 3, 4])) if causal else 0
        qp = int(g.integers(0, qP)) if qP else 0
        use_acc = bool(g.integers(0, 2)) and P > 1
        fused_layout = bool(g.integers(0, 2))
        scale = float(g.choice([0.0, 0.05, 0.2]))
        gen = torch.Generator(device=DEV).manual_seed(seed)
        buf = torch.randn(S, hq + 2 * hkv, 128, device=DEV, generator=gen).to(torch.bfloat16)
        if seed % 4 == 0:
            buf[:: max(1, S // 7), hq:hq + hkv] *= 4                   # keys that move the running maximum
        q, k, v = buf[:, :hq], buf[:, hq:hq + hkv], buf[:, hq + hkv:]
        if not fused_layout:
            q, k, v = q.contiguous(), k.contiguous(), v.contiguous()
        qf, kf, vf = q.float().contiguous(), k.float().contiguous(), v.float().contiguous()
        kw = dict(seq_len=S, chunk_start=c0, chunk_len=n, kv_len=kv_len, part_id=part, num_parts=P, part_align=align,
                  causal=causal, softmax_scale=scale, q_part_id=qp, q_num_parts=qP)
        o32 = torch.zeros(n, hq, 128, device=DEV); l32 = torch.full((n, hq), float("-inf"), device=DEV)
        acc32 = acc16 = None
        if use_acc:                                                    # state: the fp32 kernel's result over another partition
            pec.pec_prefill_attn(qf, kf, vf, o=o32, lse=l32, **{**kw, "part_id": (part + 1) % P})
            acc32, acc16 = (o32.clone(), l32.clone()), (o32.clone(), l32.clone())
        o16, l16 = o32.clone(), l32.clone()
        pec.pec_prefill_attn(qf, kf, vf, o=o32, lse=l32, acc=acc32, **kw)
        pec.pec_prefill_attn(q, k, v, o=o16, lse=l16, acc=acc16, **kw)
        pec.check_status()
        what = f"seed {seed}: S={S} hq={hq} hkv={hkv} P={P} part={part} align={align} causal={causal} c0={c0} n={n} kv={kv_len} qP={qP} qp={qp} acc={use_acc} fused={fused_layout} scale={scale}"
        fin = torch.isfinite(l32)
        assert not torch.isnan(o16).any() and not torch.isnan(l16).any(), what
        assert torch.equal(torch.isfinite(l16), fin), what
        eo = float((o16 - o32).abs().max())
        el = float((l16[fin] - l32[fin]).abs().max()) if fin.any() else 0.0
        assert eo <= 2e-2 * max(1.0, float(o32.abs().max()) / 4) and el <= 1e-3, what
        worst_o, worst_l = max(worst_o, eo), max(worst_l, el)
    print(f"[cross-check] 600 random calls, bf16 against fp32 kernel: max|dO| = {worst_o:.3e}, max|dLSE| = {worst_l:.3e}")


def test_many_random_packed_batches_with_and_without_the_worklist(pec):
    """200 seeded packed batches (1-39 requests of 0-1199 rows, now and then one of several thousand): the work-list
    changes the order of the tiles and nothing else (identical bits), and every element agrees with the fp32 kernel."""
    from paper_2409_15104_b200 import prefill
    worst_o = worst_l = 0.0
    for seed in range(200):
        g = np.random.Generator(np.random.Philox(key=888000 + seed))
        B = int(g.integers(1, 40))
        lens = [int(x) for x in g.integers(0, 1200, size=B)]
        if seed % 5 == 0:
            lens[int(g.integers(0, B))] = int(g.integers(2000, 6000))
        cu = [0] + [int(x) for x in np.cumsum(lens)]
        if cu[-1] == 0:
            continue
        hkv = int(g.choice([1, 2]))
        hq = hkv * int(g.choice([1, 4, 8]))
        gen = torch.Generator(device=DEV).manual_seed(seed)
        buf = torch.randn(cu[-1], hq + 2 * hkv, 128, device=DEV, generator=gen).to(torch.bfloat16)
        q, k, v = buf[:, :hq], buf[:, hq:hq + hkv], buf[:, hq + hkv:]
        dcu = torch.tensor(cu, dtype=torch.int32, device=DEV)
        o1, l1 = prefill.varlen_prefill(q, k, v, dcu)
        o2, l2 = prefill.varlen_prefill(q, k, v, dcu, worklist=prefill.make_worklist(cu, torch.bfloat16, DEV))
        o3, l3 = pec.pec_prefill_attn(q.float().contiguous(), k.float().contiguous(), v.float().contiguous(), cu_seqlens=dcu)
        pec.check_status()
        what = f"seed {seed}: lens={lens} hq={hq} hkv={hkv}"
        assert torch.equal(o1, o2) and torch.equal(l1, l2), what
        assert not torch.isnan(o1).any() and not torch.isnan(l1).any(), what
        eo, el = float((o1.float() - o3).abs().max()), float((l1 - l3).abs().max())
        assert eo <= 2.5e-2 and el <= 1e-3, what             # the bf16 output's own rounding on top of 2e-2
        worst_o, worst_l = max(worst_o, eo), max(worst_l, el)
    print(f"[cross-check] 200 random packed batches, bf16 against fp32 kernel: max|dO| = {worst_o:.3e}, max|dLSE| = {worst_l:.3e}")


def test_many_random_decode_calls_match_oracle(pec):
    """60 seeded decode calls: cache lengths to 20000, key ranges inside the cache (empty ones too), 1-16 query heads
    per KV head, slice counts given or chosen by the library."""
    for seed in range(60):
        g = np.random.Generator(np.random.Philox(key=999000 + seed))
        L = int(g.integers(1, 20000))
        hkv = int(g.choice([1, 2, 8]))
        grp = int(g.choice([1, 2, 4, 8, 16]))
        lo = int(g.integers(0, L)) if g.integers(0, 2) else 0
        hi = int(g.integers(lo, L + 1)) if g.integers(0, 2) else L
        splits = int(g.choice([0, 0, 1, 2, 3, 7, 16, 37]))
        k = workloads.normal_tensor(30000 + seed, 2, (L, hkv, 128), torch.bfloat16)
        v = workloads.normal_tensor(30000 + seed, 3, (L, hkv, 128), torch.bfloat16)
        q = workloads.normal_tensor(30000 + seed, 1, (hkv * grp, 128), torch.bfloat16)
        o, lse = pec.pec_decode_attn(q.to(DEV), k.to(DEV), v.to(DEV), kv_lo=lo, kv_hi=hi, num_splits=splits)
        pec.check_status()
        want = oracle.attn_rows(q[None], [L - 1], k, v, [(lo, hi)] if hi > lo else [], False)
        compare(o[None], lse[None], *want, 2e-2, 1e-3, f"decode seed {seed}: L={L} keys [{lo},{hi}) {hkv * grp}/{hkv} heads splits={splits}")
