"""Oracle entry points (test infrastructure; see pec_oracle.c for the attention arithmetic).

attention : paper Eq. 3 with the row softmax of Eq. 4 (keys up to the query's own token),
            evaluated per (row, head) in fp64 by the C routine.
merge     : the online-softmax combination of two partial results over disjoint key sets
            (Section 2.2; the colocation example's step 5 in Section 5.2 merges two such
            partial outputs of one request).
planner   : integer rules for zigzag sequence partitions, preemptible chunks and causal
            tile classes.  The paper only says that a long input is cut into segments
            (Section 2.2) and that a prefill pauses between kernels (Section 5.1); the
            concrete rule below is this library's convention, written here with Python
            integers only.
"""
import ctypes
import math

import numpy as np

from . import build as _build

SKIP, PARTIAL, FULL = 0, 1, 2

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        lib.pec_oracle_attn_rows.restype = ctypes.c_int
        lib.pec_oracle_attn_rows.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
            ctypes.c_int, ctypes.c_int, ctypes.c_int,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
            ctypes.c_int, ctypes.c_double, ctypes.c_void_p, ctypes.c_void_p,
        ]
        lib.pec_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def oracle_threads() -> int:
    """Host threads the C routine runs on."""
    return int(_load().pec_oracle_threads())


def _as_f32(x):
    """float32 C-contiguous numpy view/copy of a numpy array or a torch CPU tensor."""
    if hasattr(x, "detach"):  # torch tensor; bf16 -> fp32 is exact
        import torch
        x = x.detach().to("cpu").to(torch.float32).contiguous().numpy()
    return np.ascontiguousarray(x, dtype=np.float32)


# --------------------------------------------------------------------------- planner
def _ceil_div(a: int, b: int) -> int:
    return -((-a) // b)


def plan_partitions(seq_len, num_parts, chunk_len, align, block_m, block_n, causal, tiles=True):
    """Zigzag partitions, chunk list, tile classes and visible-pair counts (all Python ints).

    With U = ceil(S/align) alignment units, the sequence is cut into 2P blocks at
    bounds[k] = min(S, align * floor(k*U / (2P))); partition p owns blocks p and 2P-1-p,
    which pairs an early (cheap under a causal mask) block with a late (expensive) one.
    Chunk c covers query rows [c*C, min(S, (c+1)*C)).  A (query tile, key tile) pair is
    SKIP when every key lies after every query, FULL when no key lies after any query,
    PARTIAL otherwise; without the causal mask every pair is FULL.  pairs[p] counts the
    (query, key) pairs partition p's keys contribute when all S rows are queries.
    """
    S, P, C = int(seq_len), int(num_parts), int(chunk_len)
    if S < 0 or P < 1 or align < 1 or block_m < 1 or block_n < 1:
        raise ValueError("bad planner arguments")
    if C <= 0:
        C = max(S, 1)
    U = _ceil_div(S, align)
    bounds = [min(S, align * ((k * U) // (2 * P))) for k in range(2 * P + 1)]
    parts = []
    pairs = []
    for p in range(P):
        ivs = [(bounds[p], bounds[p + 1]), (bounds[2 * P - 1 - p], bounds[2 * P - p])]
        parts.append(ivs)
        n = 0
        for lo, hi in ivs:
            for j in range(lo, hi):
                n += (S - j) if causal else S
        pairs.append(n)
    n_chunks = _ceil_div(S, C)
    chunks = [(c * C, min(S, (c + 1) * C) - c * C) for c in range(n_chunks)]
    nq, nk = _ceil_div(S, block_m), _ceil_div(S, block_n)
    tile_class = None
    if tiles:
        tile_class = np.zeros((nq, nk), dtype=np.uint8)
        for a in range(nq):
            q0, q1 = a * block_m, min(S, (a + 1) * block_m)
            for b in range(nk):
                k0, k1 = b * block_n, min(S, (b + 1) * block_n)
                if not causal:
                    cls = FULL
                elif k0 > q1 - 1:
                    cls = SKIP
                elif k1 - 1 <= q0:
                    cls = FULL
                else:
                    cls = PARTIAL
                tile_class[a, b] = cls
    return {
        "bounds": bounds, "parts": parts, "pairs": pairs, "chunks": chunks,
        "nq_tiles": nq, "nk_tiles": nk, "tile_class": tile_class,
    }


def plan_worklist(cu_seqlens, block_m, block_n, causal):
    """Tile list of a packed batch of short requests (Section 5.2), heaviest first.

    Every request is cut into tiles of block_m query rows from its own first row.  A tile's weight is
    the number of block_n-key tiles of its request that hold at least one key some row of the tile can
    see: with the causal mask the tile's last row, at position e - 1, sees keys [0, e), so
    ceil(e / block_n); without it every row sees all L keys.  Entries (first row of the request, position
    of the tile's first row, rows, request length) are ordered by weight descending, then request index,
    then position."""
    cu = [int(x) for x in cu_seqlens]
    entries = []
    for b in range(len(cu) - 1):
        L = cu[b + 1] - cu[b]
        if L < 0:
            raise ValueError("cu_seqlens decreases")
        for pos0 in range(0, L, block_m):
            n = min(block_m, L - pos0)
            weight = _ceil_div(pos0 + n if causal else L, block_n)
            entries.append((-weight, b, pos0, (cu[b], pos0, n, L)))
    entries.sort(key=lambda e: e[:3])
    return [e[3] for e in entries]


def partition_rows(seq_len, num_parts, part_id, align, chunk_start=0, chunk_len=None):
    """Positions of the chunk's rows that lie in zigzag partition part_id (ascending)."""
    S = int(seq_len)
    chunk_len = S - chunk_start if chunk_len is None else int(chunk_len)
    ivs = plan_partitions(S, num_parts, 0, align, 1, 1, True, tiles=False)["parts"][part_id]
    return [i for lo, hi in ivs for i in range(max(lo, chunk_start), min(hi, chunk_start + chunk_len))]


def partition_intervals(seq_len, num_parts, part_id, align, kv_len=None):
    """Key intervals of one partition, cut to the available K/V prefix [0, kv_len)."""
    S, P, p = int(seq_len), int(num_parts), int(part_id)
    kv_len = S if kv_len is None else int(kv_len)
    if P == 1:
        ivs = [(0, S)]
    else:
        ivs = plan_partitions(S, P, 0, align, 1, 1, True, tiles=False)["parts"][p]
    out = []
    for lo, hi in ivs:
        hi = min(hi, kv_len)
        if hi > lo:
            out.append((lo, hi))
    return out


# --------------------------------------------------------------------------- attention
def attn_rows(q_rows, q_pos, k, v, intervals, causal, scale=None):
    """fp64 partial attention of the given query rows over a key set.

    q_rows [n, Hq, D]; q_pos [n] positions of those rows; k, v [n_keys, Hkv, D];
    intervals: disjoint half-open key ranges.  Returns (O [n,Hq,D] f64, LSE [n,Hq] f64).
    """
    q = _as_f32(q_rows)
    kk = _as_f32(k)
    vv = _as_f32(v)
    n, hq, d = q.shape
    n_keys, hkv, d2 = kk.shape
    assert d2 == d and vv.shape == kk.shape
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    pos = np.ascontiguousarray(q_pos, dtype=np.int64)
    assert pos.shape == (n,)
    lo = np.ascontiguousarray([a for a, _ in intervals], dtype=np.int64)
    hi = np.ascontiguousarray([b for _, b in intervals], dtype=np.int64)
    o = np.empty((n, hq, d), dtype=np.float64)
    lse = np.empty((n, hq), dtype=np.float64)
    rc = _load().pec_oracle_attn_rows(
        q.ctypes.data, pos.ctypes.data, n, kk.ctypes.data, vv.ctypes.data, n_keys,
        hq, hkv, d, lo.ctypes.data, hi.ctypes.data, len(intervals),
        1 if causal else 0, float(scale), o.ctypes.data, lse.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"pec_oracle_attn_rows failed: {rc}")
    return o, lse


def prefill_attn(q, k, v, *, seq_len, chunk_start=0, chunk_len=None, kv_len=None,
                 part_id=0, num_parts=1, part_align=128, causal=True, scale=None, rows=None):
    """What one partial-prefill call must return, for all chunk rows or for sampled ones.

    q holds the whole request's queries [seq_len, Hq, D] (indexed by position);
    k, v hold at least the first kv_len keys.  rows (optional) lists positions inside
    the chunk to evaluate; the result rows follow that list's order.
    """
    S = int(seq_len)
    chunk_len = S - chunk_start if chunk_len is None else int(chunk_len)
    kv_len = S if kv_len is None else int(kv_len)
    ivs = partition_intervals(S, num_parts, part_id, part_align, kv_len)
    if rows is None:
        pos = np.arange(chunk_start, chunk_start + chunk_len, dtype=np.int64)
    else:
        pos = np.asarray(rows, dtype=np.int64)
        assert ((pos >= chunk_start) & (pos < chunk_start + chunk_len)).all()
    if hasattr(q, "detach"):
        import torch
        q_sel = q[torch.as_tensor(pos)]
    else:
        q_sel = np.asarray(q)[pos]
    return attn_rows(q_sel, pos, k[:kv_len], v[:kv_len], ivs, causal, scale)


def varlen_attn(q, k, v, cu_seqlens, causal=True, scale=None):
    """Packed batch: request r owns rows [cu[r], cu[r+1]) and attends only to itself."""
    cu = [int(x) for x in cu_seqlens]
    qf = _as_f32(q)
    total, hq, d = qf.shape
    o = np.zeros((total, hq, d), dtype=np.float64)
    lse = np.full((total, hq), -np.inf, dtype=np.float64)
    for r in range(len(cu) - 1):
        a, b = cu[r], cu[r + 1]
        if b == a:
            continue
        pos = np.arange(b - a, dtype=np.int64)
        o[a:b], lse[a:b] = attn_rows(qf[a:b], pos, k[a:b], v[a:b], [(0, b - a)], causal, scale)
    return o, lse


# --------------------------------------------------------------------------- merge
def merge(o_a, lse_a, o_b, lse_b):
    """Combine two partial results over disjoint key sets (fp64 numpy).

    LSE = logaddexp(LSE_a, LSE_b); O = e^{LSE_a-LSE} O_a + e^{LSE_b-LSE} O_b.
    A side with LSE = -inf contributes nothing; both -inf gives (0, -inf).
    """
    o_a = np.asarray(o_a, dtype=np.float64)
    o_b = np.asarray(o_b, dtype=np.float64)
    la = np.asarray(lse_a, dtype=np.float64)
    lb = np.asarray(lse_b, dtype=np.float64)
    m = np.maximum(la, lb)
    both_empty = np.isneginf(m)
    m_safe = np.where(both_empty, 0.0, m)
    wa = np.exp(la - m_safe)
    wb = np.exp(lb - m_safe)
    tot = wa + wb
    lse = np.where(both_empty, -np.inf, m_safe + np.log(np.where(both_empty, 1.0, tot)))
    ca = np.where(both_empty, 0.0, wa / np.where(both_empty, 1.0, tot))
    cb = np.where(both_empty, 0.0, wb / np.where(both_empty, 1.0, tot))
    o = ca[..., None] * o_a + cb[..., None] * o_b
    return o, lse


def merge_n(o_parts, lse_parts):
    """Combine n partial results over pairwise disjoint key sets in one step (fp64 numpy):
    LSE = ln sum_i exp(LSE_i); O = sum_i exp(LSE_i - LSE) O_i.  Rows where every part is empty
    give (0, -inf)."""
    o_parts = [np.asarray(o, dtype=np.float64) for o in o_parts]
    ls = np.stack([np.asarray(l, dtype=np.float64) for l in lse_parts])       # [n, rows, H]
    m = ls.max(axis=0)
    empty = np.isneginf(m)
    m_safe = np.where(empty, 0.0, m)
    w = np.exp(ls - m_safe)                                                    # exp(-inf) = 0
    tot = w.sum(axis=0)
    lse = np.where(empty, -np.inf, m_safe + np.log(np.where(empty, 1.0, tot)))
    o = np.zeros_like(o_parts[0])
    for i, oi in enumerate(o_parts):
        c = np.where(empty, 0.0, w[i] / np.where(empty, 1.0, tot))
        o += c[..., None] * np.where(c[..., None] == 0.0, 0.0, oi)
    return o, lse


# --------------------------------------------------------------------------- SP strategy cost model
def ring_segments(seq_len, num_parts, align, layout):
    """Row intervals of every ring rank's segment: layout "zigzag" pairs block r with block 2P-1-r of
    2P equal blocks, layout "contiguous" cuts P blocks; block bounds are align * floor(k*U/nblocks)
    with U = ceil(S/align), cut at S."""
    S, P = int(seq_len), int(num_parts)
    U = _ceil_div(S, align)
    if layout == "zigzag":
        b = [min(S, align * ((k * U) // (2 * P))) for k in range(2 * P + 1)]
        return [[(b[r], b[r + 1]), (b[2 * P - 1 - r], b[2 * P - r])] for r in range(P)]
    if layout == "contiguous":
        b = [min(S, align * ((k * U) // P)) for k in range(P + 1)]
        return [[(b[r], b[r + 1])] for r in range(P)]
    raise ValueError("unknown layout")


def plan_ring(seq_len, num_parts, align, layout, causal):
    """Work of ring-attention sequence parallelism (Section 2.2), counted row by row.

    Rank r keeps the query rows of its segment; at step t it holds the keys of the segment of rank
    (r - t) mod P.  pairs[r][t] = sum over the rank's rows i of the number of those keys visible to
    row i (keys j <= i under the causal mask, else all of them).  step_max[t] = max over ranks,
    rank_total[r] = sum over steps.
    """
    S, P = int(seq_len), int(num_parts)
    if S < 0 or P < 1 or align < 1:
        raise ValueError("bad planner arguments")
    seg = ring_segments(S, P, align, layout)
    pairs = [[0] * P for _ in range(P)]
    for r in range(P):
        for t in range(P):
            keys = seg[(r - t) % P]
            n = 0
            for q_lo, q_hi in seg[r]:
                for i in range(q_lo, q_hi):
                    for k_lo, k_hi in keys:
                        last = min(k_hi, i + 1) if causal else k_hi     # exclusive end of the visible keys
                        n += max(0, last - k_lo)
            pairs[r][t] = n
    return {"pairs": pairs,
            "step_max": [max(pairs[r][t] for r in range(P)) for t in range(P)],
            "rank_total": [sum(pairs[r]) for r in range(P)]}


def balance_batches(lengths, replicas):
    """Token-balanced short-request batches (Section 5.2 states the goal only).  Rule: take the
    requests longest first (equal lengths in index order) and give each to the replica with the
    fewest tokens so far (equal totals: the lowest id).  Returns (assign, tokens)."""
    if replicas < 1 or any(x < 0 for x in lengths):
        raise ValueError("bad arguments")
    tokens = [0] * replicas
    assign = [None] * len(lengths)
    remaining = list(range(len(lengths)))
    while remaining:
        longest = max(lengths[i] for i in remaining)
        i = next(i for i in remaining if lengths[i] == longest)
        remaining.remove(i)
        rep = tokens.index(min(tokens))
        assign[i] = rep
        tokens[rep] += lengths[i]
    return assign, tokens


def sp_volumes(s, d, n_h, n_kv, d_h, T, G):
    """Section 5.3's communication (per node) and computation (per GPU) volumes, written term by term
    with exact rational arithmetic: {(stage, strategy): (comm, comp)} for stage in ("attn", "mlp") and
    strategy in ("megatron", "ulysses")."""
    from fractions import Fraction as F
    s, d, n_h, n_kv, d_h, T, G = (F(x) for x in (s, d, n_h, n_kv, d_h, T, G))
    qkv = 2 * s * d * (n_h + n_kv) * d_h          # QKV generation on a full segment
    out_proj = 2 * s * d * d                      # post-self-attention linear
    vols = {}
    # attention stage, Megatron SP: all-gather + reduce-scatter; QKV split over T, attention over s*T tokens / T
    vols[("attn", "megatron")] = (2 * s * d * (T - 1) * G, qkv / T + 4 * (s * T) ** 2 * d / T + out_proj)
    # attention stage, Ulysses SP: two all-to-alls + parameter transfer; attention over s*G tokens / G
    a2a = 2 * s * (n_h + n_kv) * d_h * (G - 1)
    params = (d * (n_h + n_kv) * d_h + d * d) * G * (T - 1) / T
    vols[("attn", "ulysses")] = (a2a + params, qkv + 4 * (s * G) ** 2 * d / G + out_proj)
    # MLP stage: 16 s d^2 either way; Megatron moves embeddings, Ulysses moves the 8 d^2 parameters
    vols[("mlp", "megatron")] = (2 * s * d * (T - 1) * G, 16 * s * d * d)
    vols[("mlp", "ulysses")] = (8 * d * d * (T - 1) * G / T, 16 * s * d * d)
    return vols


def select_sp(s, d, n_h, n_kv, d_h, T, G, elem_bytes, node_bw, gpu_flops):
    """The combination with the lowest estimated latency (comm bytes / node_bw + comp / gpu_flops);
    ties go to Megatron.  Returns ((attn, mlp), {combo: seconds})."""
    from fractions import Fraction as F
    vols = sp_volumes(s, d, n_h, n_kv, d_h, T, G)
    times = {}
    for a in ("megatron", "ulysses"):
        for m in ("megatron", "ulysses"):
            comm = vols[("attn", a)][0] + vols[("mlp", m)][0]
            comp = vols[("attn", a)][1] + vols[("mlp", m)][1]
            times[(a, m)] = comm * F(elem_bytes) / F(node_bw) + comp / F(gpu_flops)
    order = [("megatron", "megatron"), ("megatron", "ulysses"), ("ulysses", "megatron"), ("ulysses", "ulysses")]
    best = min(order, key=lambda c: (times[c], order.index(c)))
    return best, times


# --------------------------------------------------------------------------- dense steps (Eq. 2, Eq. 5)
def linear(x, w):
    """y = x w^T in fp64 (numpy matmul): QKV generation (Eq. 2) with the per-head weights stacked
    row-wise in w, or the post-self-attention linear layer (Eq. 5) with w = W_L^T."""
    return _as_f32(x).astype(np.float64) @ _as_f32(w).astype(np.float64).T


def rope(y, positions, theta, rot_cols, head_dim=128):
    """Rotary position encoding of the leading rot_cols columns of y [T, N] (fp64 numpy).  The paper
    never states a position encoding; the Llama models it serves (Section 6.1) use the rotary form of
    RoFormer in its "rotate-half" pairing, which is what this restates: the columns are heads of
    head_dim channels, channel i < head_dim/2 of a head pairs with channel i + head_dim/2, and the
    pair of the token at position p is turned by the angle p * theta**(-2 i / head_dim):
        out[i]       = y[i] cos - y[i + d/2] sin
        out[i + d/2] = y[i + d/2] cos + y[i] sin.
    Columns from rot_cols on (the values) are returned unchanged."""
    out = _as_f32(y).astype(np.float64) if hasattr(y, "detach") else np.array(y, dtype=np.float64, copy=True)
    pos = np.asarray(positions, dtype=np.float64).reshape(-1)
    assert out.shape[0] == pos.shape[0] and rot_cols % head_dim == 0 and rot_cols <= out.shape[1]
    half = head_dim // 2
    inv_freq = np.float64(theta) ** (-2.0 * np.arange(half, dtype=np.float64) / head_dim)
    ang = pos[:, None] * inv_freq[None, :]                                     # [T, d/2]
    c, s_ = np.cos(ang), np.sin(ang)
    for h0 in range(0, rot_cols, head_dim):
        a = out[:, h0:h0 + half].copy()
        b = out[:, h0 + half:h0 + head_dim].copy()
        out[:, h0:h0 + half] = a * c - b * s_
        out[:, h0 + half:h0 + head_dim] = b * c + a * s_
    return out


def linear_rope(x, w, positions, theta, rot_cols, head_dim=128):
    """QKV generation (Eq. 2) followed by the rotary encoding of the query and key heads."""
    return rope(linear(x, w), positions, theta, rot_cols, head_dim)

