"""ctypes binding of libpec.so.  Argument marshalling only: every step runs in the library.

Function names mirror the C ABI (include/pec.h).  torch provides device memory and streams.
The library is loaded on first use; a missing or unloadable library raises - there is no
fallback implementation.
"""
import ctypes
import os

import torch

PEC_OK = 0
PEC_ERR_TIMEOUT = -6
PEC_BF16, PEC_F32 = 1, 2
PEC_TILE_SKIP, PEC_TILE_PARTIAL, PEC_TILE_FULL = 0, 1, 2
PEC_LAYOUT_ZIGZAG, PEC_LAYOUT_CONTIGUOUS = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpec.so")
_lib = None
_status_words = {}


class PecError(RuntimeError):
    def __init__(self, code, text):
        super().__init__(f"pec error {code}: {text}")
        self.code = code


class pec_attn_args(ctypes.Structure):
    _fields_ = [
        ("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p),
        ("q_stride_t", ctypes.c_int64), ("q_stride_h", ctypes.c_int64),
        ("k_stride_t", ctypes.c_int64), ("k_stride_h", ctypes.c_int64),
        ("v_stride_t", ctypes.c_int64), ("v_stride_h", ctypes.c_int64),
        ("in_dtype", ctypes.c_int32),
        ("o", ctypes.c_void_p), ("o_dtype", ctypes.c_int32),
        ("lse", ctypes.c_void_p),
        ("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("D", ctypes.c_int32),
        ("cu_seqlens", ctypes.c_void_p), ("B", ctypes.c_int32),
        ("seq_len", ctypes.c_int64),
        ("chunk_start", ctypes.c_int64), ("chunk_len", ctypes.c_int64),
        ("kv_len", ctypes.c_int64),
        ("part_id", ctypes.c_int32), ("num_parts", ctypes.c_int32),
        ("part_align", ctypes.c_int32), ("causal", ctypes.c_int32),
        ("softmax_scale", ctypes.c_float),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
        ("status", ctypes.c_void_p),
        ("acc_o", ctypes.c_void_p), ("acc_lse", ctypes.c_void_p),
        ("q_part_id", ctypes.c_int32), ("q_num_parts", ctypes.c_int32),
        ("worklist", ctypes.c_void_p), ("n_items", ctypes.c_int32), ("worklist_block_m", ctypes.c_int32),
        ("overlap_previous", ctypes.c_int32),
    ]


class pec_decode_args(ctypes.Structure):
    _fields_ = [
        ("q", ctypes.c_void_p), ("q_stride_h", ctypes.c_int64),
        ("k", ctypes.c_void_p), ("v", ctypes.c_void_p),
        ("k_stride_t", ctypes.c_int64), ("k_stride_h", ctypes.c_int64),
        ("v_stride_t", ctypes.c_int64), ("v_stride_h", ctypes.c_int64),
        ("o", ctypes.c_void_p), ("o_dtype", ctypes.c_int32), ("lse", ctypes.c_void_p),
        ("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("D", ctypes.c_int32),
        ("kv_lo", ctypes.c_int64), ("kv_hi", ctypes.c_int64),
        ("num_splits", ctypes.c_int32), ("softmax_scale", ctypes.c_float),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
        ("status", ctypes.c_void_p),
    ]


class pec_sp_inputs(ctypes.Structure):
    _fields_ = [(n, ctypes.c_double) for n in ("s", "d", "n_h", "n_kv", "d_h", "T", "G", "elem_bytes", "node_bw", "gpu_flops")]


class pec_sp_choice(ctypes.Structure):
    _fields_ = [("attn_strategy", ctypes.c_int32), ("mlp_strategy", ctypes.c_int32),
                ("comm", (ctypes.c_double * 2) * 2), ("comp", (ctypes.c_double * 2) * 2), ("seconds", ctypes.c_double * 4)]


class pec_plan(ctypes.Structure):
    _fields_ = [
        ("bounds", ctypes.POINTER(ctypes.c_int64)), ("bounds_cap", ctypes.c_int64),
        ("part_lo", ctypes.POINTER(ctypes.c_int64)), ("part_hi", ctypes.POINTER(ctypes.c_int64)),
        ("part_cap", ctypes.c_int64),
        ("pairs", ctypes.POINTER(ctypes.c_int64)), ("pairs_cap", ctypes.c_int64),
        ("chunk_start", ctypes.POINTER(ctypes.c_int64)), ("chunk_len", ctypes.POINTER(ctypes.c_int64)),
        ("chunk_cap", ctypes.c_int64),
        ("tile_class", ctypes.POINTER(ctypes.c_uint8)), ("tile_cap", ctypes.c_int64),
        ("n_bounds", ctypes.c_int64), ("n_parts", ctypes.c_int64), ("n_chunks", ctypes.c_int64),
        ("nq_tiles", ctypes.c_int64), ("nk_tiles", ctypes.c_int64),
    ]


EXPORTS = ("pec_prefill_attn", "pec_workspace_size", "pec_attn_merge", "pec_attn_merge_n", "pec_plan_partitions",
           "pec_last_error", "pec_decode_attn", "pec_decode_workspace_size", "pec_decode_attn_static", "pec_select_sp", "pec_linear",
           "pec_plan_ring", "pec_balance_batches", "pec_plan_worklist", "pec_worklist_block_m", "pec_control",
           "pec_linear_merged", "pec_linear_rope", "pec_rope_table", "pec_rope_table_floats")
PEC_CTL_WAIT_LIMIT_CYCLES, PEC_CTL_TEST_SKIP_LAST_LOAD = 1, 2
PEC_DECODE_STATIC_SCRATCH_BYTES = 4 * 1024 * 1024
PEC_MERGE_MAX_PARTS = 16
PEC_LINEAR_MERGED_MAX_PARTS = 8


def load():
    """Load libpec.so (building is a separate step: python -m paper_2409_15104_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2409_15104_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    lib.pec_prefill_attn.restype = ctypes.c_int
    lib.pec_prefill_attn.argtypes = [ctypes.POINTER(pec_attn_args), ctypes.c_void_p]
    lib.pec_workspace_size.restype = ctypes.c_size_t
    lib.pec_workspace_size.argtypes = [ctypes.POINTER(pec_attn_args)]
    lib.pec_attn_merge.restype = ctypes.c_int
    lib.pec_attn_merge.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                   ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32,
                                   ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p]
    lib.pec_attn_merge_n.restype = ctypes.c_int
    lib.pec_attn_merge_n.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_void_p), ctypes.c_int32,
                                     ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32,
                                     ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p]
    lib.pec_plan_partitions.restype = ctypes.c_int
    lib.pec_plan_partitions.argtypes = [ctypes.c_int64, ctypes.c_int32, ctypes.c_int64, ctypes.c_int32,
                                        ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(pec_plan)]
    lib.pec_decode_attn.restype = ctypes.c_int
    lib.pec_decode_attn.argtypes = [ctypes.POINTER(pec_decode_args), ctypes.c_void_p]
    lib.pec_decode_attn_static.restype = ctypes.c_int
    lib.pec_decode_attn_static.argtypes = [ctypes.POINTER(pec_decode_args), ctypes.c_void_p]
    lib.pec_decode_workspace_size.restype = ctypes.c_size_t
    lib.pec_decode_workspace_size.argtypes = [ctypes.POINTER(pec_decode_args)]
    lib.pec_linear.restype = ctypes.c_int
    lib.pec_linear.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                               ctypes.c_int64, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p,
                               ctypes.c_void_p]
    lib.pec_linear_rope.restype = ctypes.c_int
    lib.pec_linear_rope.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                                    ctypes.c_int64, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p,
                                    ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32,
                                    ctypes.c_void_p, ctypes.c_void_p]
    lib.pec_rope_table.restype = ctypes.c_int
    lib.pec_rope_table.argtypes = [ctypes.c_double, ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
    lib.pec_rope_table_floats.restype = ctypes.c_size_t
    lib.pec_rope_table_floats.argtypes = [ctypes.c_int64]
    lib.pec_linear_merged.restype = ctypes.c_int
    lib.pec_linear_merged.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_void_p), ctypes.c_int32,
                                      ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int64,
                                      ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
    lib.pec_select_sp.restype = ctypes.c_int
    lib.pec_select_sp.argtypes = [ctypes.POINTER(pec_sp_inputs), ctypes.POINTER(pec_sp_choice)]
    lib.pec_plan_ring.restype = ctypes.c_int
    lib.pec_plan_ring.argtypes = [ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                  ctypes.POINTER(ctypes.c_int64), ctypes.c_int64, ctypes.POINTER(ctypes.c_int64),
                                  ctypes.POINTER(ctypes.c_int64), ctypes.c_int64]
    lib.pec_balance_batches.restype = ctypes.c_int
    lib.pec_balance_batches.argtypes = [ctypes.POINTER(ctypes.c_int32), ctypes.c_int32, ctypes.c_int32,
                                        ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int64)]
    lib.pec_plan_worklist.restype = ctypes.c_int
    lib.pec_plan_worklist.argtypes = [ctypes.POINTER(ctypes.c_int32), ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                      ctypes.c_int32, ctypes.POINTER(ctypes.c_int32), ctypes.c_int64,
                                      ctypes.POINTER(ctypes.c_int64)]
    lib.pec_worklist_block_m.restype = ctypes.c_int32
    lib.pec_worklist_block_m.argtypes = [ctypes.c_int32]
    lib.pec_control.restype = ctypes.c_int
    lib.pec_control.argtypes = [ctypes.c_int32, ctypes.c_int64]
    lib.pec_last_error.restype = ctypes.c_char_p
    lib.pec_last_error.argtypes = []
    _lib = lib
    return lib


def pec_last_error() -> str:
    return load().pec_last_error().decode()


def _check(rc):
    if rc != PEC_OK:
        raise PecError(rc, pec_last_error())


def _dtype_code(dt):
    if dt == torch.bfloat16:
        return PEC_BF16
    if dt == torch.float32:
        return PEC_F32
    raise TypeError(f"unsupported dtype {dt}")


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def status_word(device=None) -> torch.Tensor:
    """The per-device int32 word kernels flag expired waits in (zero = fine)."""
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    key = dev.index if dev.index is not None else torch.cuda.current_device()
    if key not in _status_words:
        _status_words[key] = torch.zeros(1, dtype=torch.int32, device=dev)
    return _status_words[key]


def check_status(device=None):
    """Synchronise and raise if a kernel recorded an expired wait; clears the word."""
    w = status_word(device)
    code = int(w.item())
    if code != 0:
        w.zero_()
        raise PecError(code, "a kernel's bounded wait expired" if code == PEC_ERR_TIMEOUT else "kernel status")


def pec_prefill_attn(q, k, v, *, seq_len=None, chunk_start=0, chunk_len=None, kv_len=None,
                     part_id=0, num_parts=1, part_align=128, causal=True, softmax_scale=0.0,
                     cu_seqlens=None, out_dtype=None, o=None, lse=None, stream=None,
                     acc=None, q_part_id=0, q_num_parts=0, worklist=None, overlap_previous=False):
    """Partial attention of one chunk / partition / packed batch; returns (o, lse).

    q [T, Hq, 128], k / v [Tk, Hkv, 128] CUDA tensors (last dim contiguous).  Single request:
    rows are positions, the call covers query rows [chunk_start, chunk_start+chunk_len) against
    keys [0, kv_len).  Packed batch: pass cu_seqlens (int32 CUDA tensor [B+1]).
    o / lse may be passed in (views are fine as long as they are contiguous).
    acc = (o, lse) fp32 tensors: an incoming state of the same rows that the call merges its result
    into (pass the same tensors as o / lse for an in-place chain).  q_num_parts > 1 restricts the
    query rows to zigzag partition q_part_id.  worklist: int32 CUDA tensor [n, 4] from
    pec_plan_worklist (packed batches).  overlap_previous=True: the inputs were complete before the kernel that
    precedes this call on the stream, so the call may start while that kernel's last CTAs finish.
    """
    lib = load()
    assert q.is_cuda and k.is_cuda and v.is_cuda
    assert q.stride(2) == 1 and k.stride(2) == 1 and v.stride(2) == 1
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    if cu_seqlens is not None:
        B = cu_seqlens.numel() - 1
        seq_len = T if seq_len is None else seq_len
        chunk_len = seq_len
        kv_len = seq_len
    else:
        B = 1
        seq_len = T if seq_len is None else seq_len
        chunk_len = seq_len - chunk_start if chunk_len is None else chunk_len
        kv_len = (chunk_start + chunk_len if causal else seq_len) if kv_len is None else kv_len
    out_dtype = (torch.float32 if num_parts > 1 else q.dtype) if out_dtype is None else out_dtype
    if o is None:
        o = torch.empty((chunk_len, Hq, D), dtype=out_dtype, device=q.device)
    if lse is None:
        lse = torch.empty((chunk_len, Hq), dtype=torch.float32, device=q.device)
    assert o.is_contiguous() and lse.is_contiguous() and lse.dtype == torch.float32
    a = pec_attn_args()
    a.q, a.k, a.v = q.data_ptr(), k.data_ptr(), v.data_ptr()
    a.q_stride_t, a.q_stride_h = q.stride(0), q.stride(1)
    a.k_stride_t, a.k_stride_h = k.stride(0), k.stride(1)
    a.v_stride_t, a.v_stride_h = v.stride(0), v.stride(1)
    a.in_dtype = _dtype_code(q.dtype)
    a.o, a.o_dtype, a.lse = o.data_ptr(), _dtype_code(o.dtype), lse.data_ptr()
    a.Hq, a.Hkv, a.D = Hq, Hkv, D
    a.cu_seqlens = cu_seqlens.data_ptr() if cu_seqlens is not None else None
    a.B = B
    a.seq_len, a.chunk_start, a.chunk_len, a.kv_len = seq_len, chunk_start, chunk_len, kv_len
    a.part_id, a.num_parts, a.part_align = part_id, num_parts, part_align
    a.causal = 1 if causal else 0
    a.softmax_scale = float(softmax_scale)
    a.workspace, a.workspace_bytes = None, 0
    a.status = status_word(q.device).data_ptr()
    if acc is not None:
        acc_o, acc_l = acc
        assert acc_o.is_contiguous() and acc_l.is_contiguous() and acc_o.dtype == torch.float32 and acc_l.dtype == torch.float32
        assert acc_o.shape == (chunk_len, Hq, D) and acc_l.shape == (chunk_len, Hq)
        a.acc_o, a.acc_lse = acc_o.data_ptr(), acc_l.data_ptr()
    a.q_part_id, a.q_num_parts = q_part_id, q_num_parts
    a.overlap_previous = 1 if overlap_previous else 0
    if worklist is not None:
        assert worklist.is_cuda and worklist.dtype == torch.int32 and worklist.is_contiguous()
        a.worklist, a.n_items = worklist.data_ptr(), worklist.shape[0]
        a.worklist_block_m = int(lib.pec_worklist_block_m(a.in_dtype))
    _check(lib.pec_prefill_attn(ctypes.byref(a), _stream_ptr(stream)))
    return o, lse


def pec_workspace_size(**kw) -> int:
    a = pec_attn_args()
    for key, val in kw.items():
        setattr(a, key, val)
    return int(load().pec_workspace_size(ctypes.byref(a)))


def pec_attn_merge(o_a, lse_a, o_b, lse_b, *, out_dtype=torch.float32, o_out=None, lse_out=None,
                   inplace=False, stream=None):
    """Merge two fp32 partials of the same rows; returns (o, lse).  inplace=True writes into side a."""
    lib = load()
    rows, Hq, D = o_a.shape
    for t in (o_a, lse_a, o_b, lse_b):
        assert t.is_cuda and t.is_contiguous()
    if inplace:
        o_out, lse_out = o_a, lse_a
    if o_out is None:
        o_out = torch.empty((rows, Hq, D), dtype=out_dtype, device=o_a.device)
    if lse_out is None:
        lse_out = torch.empty((rows, Hq), dtype=torch.float32, device=o_a.device)
    _check(lib.pec_attn_merge(o_a.data_ptr(), lse_a.data_ptr(), o_b.data_ptr(), lse_b.data_ptr(),
                              o_out.data_ptr(), lse_out.data_ptr(), rows, Hq, D,
                              _dtype_code(o_a.dtype), _dtype_code(o_out.dtype), _stream_ptr(stream)))
    return o_out, lse_out


def pec_attn_merge_n(o_parts, lse_parts, *, out_dtype=torch.float32, o_out=None, lse_out=None, inplace=False,
                     stream=None):
    """Merge n fp32 partials of the same rows in one pass; returns (o, lse).  inplace=True writes into part 0."""
    lib = load()
    n = len(o_parts)
    assert n == len(lse_parts)
    rows, Hq, D = o_parts[0].shape
    for t in list(o_parts) + list(lse_parts):
        assert t.is_cuda and t.is_contiguous()
    if inplace:
        o_out, lse_out = o_parts[0], lse_parts[0]
    if o_out is None:
        o_out = torch.empty((rows, Hq, D), dtype=out_dtype, device=o_parts[0].device)
    if lse_out is None:
        lse_out = torch.empty((rows, Hq), dtype=torch.float32, device=o_parts[0].device)
    op = (ctypes.c_void_p * n)(*[t.data_ptr() for t in o_parts])
    lp = (ctypes.c_void_p * n)(*[t.data_ptr() for t in lse_parts])
    _check(lib.pec_attn_merge_n(op, lp, n, o_out.data_ptr(), lse_out.data_ptr(), rows, Hq, D,
                                _dtype_code(o_parts[0].dtype), _dtype_code(o_out.dtype), _stream_ptr(stream)))
    return o_out, lse_out


def decode_args(q, k, v, o, lse, kv_lo, kv_hi, num_splits=0, softmax_scale=0.0):
    """Fill a pec_decode_args from tensors (q [Hq,128], k/v [Tk,Hkv,128], o [Hq,128], lse [Hq])."""
    a = pec_decode_args()
    a.q, a.q_stride_h = q.data_ptr(), q.stride(0)
    a.k, a.v = k.data_ptr(), v.data_ptr()
    a.k_stride_t, a.k_stride_h = k.stride(0), k.stride(1)
    a.v_stride_t, a.v_stride_h = v.stride(0), v.stride(1)
    a.o, a.o_dtype, a.lse = o.data_ptr(), _dtype_code(o.dtype), lse.data_ptr()
    a.Hq, a.Hkv, a.D = q.shape[0], k.shape[1], q.shape[1]
    a.kv_lo, a.kv_hi = kv_lo, kv_hi
    a.num_splits, a.softmax_scale = num_splits, float(softmax_scale)
    a.workspace, a.workspace_bytes = None, 0
    a.status = status_word(q.device).data_ptr()
    return a


def pec_decode_workspace_size(a) -> int:
    return int(load().pec_decode_workspace_size(ctypes.byref(a)))


def pec_decode_attn(q, k, v, *, kv_lo=0, kv_hi=None, num_splits=0, softmax_scale=0.0, out_dtype=torch.float32,
                    o=None, lse=None, workspace=None, stream=None):
    """One GPU's share of a long request's decode step: the new token's attention over keys
    [kv_lo, kv_hi) of its K/V cache; returns (o [Hq,128], lse [Hq]).  The workspace tensor (uint8,
    CUDA) is allocated here when not given."""
    lib = load()
    assert q.is_cuda and q.dtype == torch.bfloat16 and q.stride(1) == 1 and k.stride(2) == 1 and v.stride(2) == 1
    kv_hi = k.shape[0] if kv_hi is None else kv_hi
    if o is None:
        o = torch.empty((q.shape[0], 128), dtype=out_dtype, device=q.device)
    if lse is None:
        lse = torch.empty((q.shape[0],), dtype=torch.float32, device=q.device)
    a = decode_args(q, k, v, o, lse, kv_lo, kv_hi, num_splits, softmax_scale)
    need = pec_decode_workspace_size(a)
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=q.device)
    a.workspace, a.workspace_bytes = workspace.data_ptr(), workspace.numel()
    _check(lib.pec_decode_attn(ctypes.byref(a), _stream_ptr(stream)))
    return o, lse


def pec_linear(x, w, y=None, stream=None):
    """y = x w^T (bf16, fp32 accumulation); x [M,K], w [N,K] CUDA tensors with contiguous rows; returns y [M,N]."""
    lib = load()
    assert x.is_cuda and w.is_cuda and x.dtype == torch.bfloat16 and w.dtype == torch.bfloat16
    assert x.stride(1) == 1 and w.stride(1) == 1 and x.shape[1] == w.shape[1]
    M, K = x.shape
    N = w.shape[0]
    if y is None:
        y = torch.empty((M, N), dtype=torch.bfloat16, device=x.device)
    assert y.stride(1) == 1
    _check(lib.pec_linear(x.data_ptr(), x.stride(0), w.data_ptr(), w.stride(0), y.data_ptr(), y.stride(0), M, N, K,
                          status_word(x.device).data_ptr(), _stream_ptr(stream)))
    return y


def pec_rope_table(theta, n_pos, device, stream=None):
    """The rotary-encoding table for positions 0 .. n_pos - 1 (head_dim 128): (tensor, n_pos), as pec_linear_rope takes it."""
    lib = load()
    table = torch.empty((lib.pec_rope_table_floats(n_pos),), dtype=torch.float32, device=device)
    _check(lib.pec_rope_table(float(theta), n_pos, 128, table.data_ptr(), _stream_ptr(stream)))
    return table, n_pos


def rope_table_angles(tables):
    """(cos, sin) [n_pos, 64] in fp64 as the kernel combines them from the table's fp32 entries (for inspection and tests)."""
    table, n_pos = tables
    t = table.double().cpu()
    na = (n_pos + 63) // 64
    F, G = t[:4096].view(64, 64), t[4096:8192].view(64, 64)            # [i][b]
    C, S = t[8192:8192 + na * 64].view(na, 64), t[8192 + na * 64:].view(na, 64)
    p = torch.arange(n_pos)
    a, b = p // 64, p % 64
    cos = C[a] * F.T[b] - S[a] * G.T[b]
    sin = S[a] * F.T[b] + C[a] * G.T[b]
    return cos, sin


def pec_linear_rope(x, w, tables, rot_cols, *, positions=None, pos0=0, y=None, stream=None):
    """y = x w^T with the rotary encoding of the leading rot_cols columns (whole heads of 128); tables = pec_rope_table(...).
    positions: int32 CUDA tensor [M] (packed batches) or None: row r is at position pos0 + r."""
    lib = load()
    table, n_pos = tables
    assert x.is_cuda and w.is_cuda and x.dtype == torch.bfloat16 and w.dtype == torch.bfloat16
    assert x.stride(1) == 1 and w.stride(1) == 1 and x.shape[1] == w.shape[1]
    assert table.is_cuda and table.is_contiguous() and table.dtype == torch.float32
    M, K = x.shape
    N = w.shape[0]
    if y is None:
        y = torch.empty((M, N), dtype=torch.bfloat16, device=x.device)
    assert y.stride(1) == 1
    if positions is not None:
        assert positions.is_cuda and positions.dtype == torch.int32 and positions.is_contiguous() and positions.numel() == M
    _check(lib.pec_linear_rope(x.data_ptr(), x.stride(0), w.data_ptr(), w.stride(0), y.data_ptr(), y.stride(0), M, N, K,
                               table.data_ptr(), n_pos, positions.data_ptr() if positions is not None else None, pos0,
                               rot_cols, status_word(x.device).data_ptr(), _stream_ptr(stream)))
    return y


def pec_linear_merged(o_parts, lse_parts, w, y=None, stream=None):
    """y = merge(o_parts, lse_parts) w^T: fp32 partials [rows,Hq,128] with LSEs [rows,Hq], w [N,Hq*128] bf16; returns y [rows,N] bf16."""
    lib = load()
    n = len(o_parts)
    assert n == len(lse_parts)
    rows, Hq, D = o_parts[0].shape
    for t in list(o_parts) + list(lse_parts):
        assert t.is_cuda and t.is_contiguous() and t.dtype == torch.float32
    assert w.is_cuda and w.dtype == torch.bfloat16 and w.stride(1) == 1 and w.shape[1] == Hq * D
    N = w.shape[0]
    if y is None:
        y = torch.empty((rows, N), dtype=torch.bfloat16, device=w.device)
    assert y.stride(1) == 1
    op = (ctypes.c_void_p * n)(*[t.data_ptr() for t in o_parts])
    lp = (ctypes.c_void_p * n)(*[t.data_ptr() for t in lse_parts])
    _check(lib.pec_linear_merged(op, lp, n, rows, Hq, D, w.data_ptr(), w.stride(0), y.data_ptr(), y.stride(0), N,
                                 status_word(w.device).data_ptr(), _stream_ptr(stream)))
    return y


def pec_select_sp(s, d, n_h, n_kv, d_h, T, G, elem_bytes=2.0, node_bw=1.0, gpu_flops=1.0):
    """Section 5.3's strategy choice; returns a dict (strategies: 0 = Megatron SP, 1 = Ulysses SP)."""
    lib = load()
    i = pec_sp_inputs(s, d, n_h, n_kv, d_h, T, G, elem_bytes, node_bw, gpu_flops)
    o = pec_sp_choice()
    _check(lib.pec_select_sp(ctypes.byref(i), ctypes.byref(o)))
    return {"attn_strategy": o.attn_strategy, "mlp_strategy": o.mlp_strategy,
            "comm": [[o.comm[a][b] for b in range(2)] for a in range(2)],
            "comp": [[o.comp[a][b] for b in range(2)] for a in range(2)],
            "seconds": [o.seconds[i] for i in range(4)]}


def pec_plan_partitions(seq_len, num_parts, chunk_len=0, align=128, block_m=128, block_n=128,
                        causal=True, tiles=True):
    """Host plan (see include/pec.h) as a dict of Python ints / a numpy uint8 tile-class array."""
    import numpy as np
    lib = load()
    plan = pec_plan()
    _check(lib.pec_plan_partitions(seq_len, num_parts, chunk_len, align, block_m, block_n, 1 if causal else 0,
                                   ctypes.byref(plan)))
    P, nch = plan.n_parts, plan.n_chunks
    bounds = (ctypes.c_int64 * plan.n_bounds)()
    lo = (ctypes.c_int64 * (2 * P))()
    hi = (ctypes.c_int64 * (2 * P))()
    pairs = (ctypes.c_int64 * P)()
    cs = (ctypes.c_int64 * max(nch, 1))()
    cl = (ctypes.c_int64 * max(nch, 1))()
    plan.bounds, plan.bounds_cap = bounds, plan.n_bounds
    plan.part_lo, plan.part_hi, plan.part_cap = lo, hi, 2 * P
    plan.pairs, plan.pairs_cap = pairs, P
    plan.chunk_start, plan.chunk_len, plan.chunk_cap = cs, cl, max(nch, 1)
    tc = None
    if tiles:
        tc = np.zeros((plan.nq_tiles, plan.nk_tiles), dtype=np.uint8)
        plan.tile_class = tc.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8))
        plan.tile_cap = tc.size
    _check(lib.pec_plan_partitions(seq_len, num_parts, chunk_len, align, block_m, block_n, 1 if causal else 0,
                                   ctypes.byref(plan)))
    return {
        "bounds": [int(x) for x in bounds],
        "parts": [[(int(lo[2 * p]), int(hi[2 * p])), (int(lo[2 * p + 1]), int(hi[2 * p + 1]))] for p in range(P)],
        "pairs": [int(x) for x in pairs],
        "chunks": [(int(cs[c]), int(cl[c])) for c in range(nch)],
        "nq_tiles": int(plan.nq_tiles), "nk_tiles": int(plan.nk_tiles), "tile_class": tc,
    }


def pec_plan_worklist(cu_seqlens, block_m, block_n=128, causal=True):
    """Heaviest-first tile list of a packed batch (see include/pec.h) as a numpy int32 array [n, 4];
    cu_seqlens is a host sequence of B + 1 offsets."""
    import numpy as np
    lib = load()
    cu = (ctypes.c_int32 * len(cu_seqlens))(*[int(x) for x in cu_seqlens])
    B = len(cu_seqlens) - 1
    n = ctypes.c_int64(0)
    _check(lib.pec_plan_worklist(cu, B, block_m, block_n, 1 if causal else 0, None, 0, ctypes.byref(n)))
    items = np.zeros((max(n.value, 1), 4), dtype=np.int32)
    _check(lib.pec_plan_worklist(cu, B, block_m, block_n, 1 if causal else 0,
                                 items.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), items.shape[0], ctypes.byref(n)))
    return items[:n.value]


def pec_worklist_block_m(dtype) -> int:
    return int(load().pec_worklist_block_m(_dtype_code(dtype)))


def pec_control(what, value):
    _check(load().pec_control(what, value))


def pec_plan_ring(seq_len, num_parts, align=128, layout=PEC_LAYOUT_ZIGZAG, causal=True):
    """Ring-attention work plan (see include/pec.h): pairs[r][t], step_max[t], rank_total[r] as Python ints."""
    lib = load()
    P = num_parts
    pairs = (ctypes.c_int64 * max(P * P, 1))()
    step_max = (ctypes.c_int64 * max(P, 1))()
    rank_total = (ctypes.c_int64 * max(P, 1))()
    _check(lib.pec_plan_ring(seq_len, num_parts, align, layout, 1 if causal else 0, pairs, max(P * P, 1),
                             step_max, rank_total, max(P, 1)))
    return {"pairs": [[int(pairs[r * P + t]) for t in range(P)] for r in range(P)],
            "step_max": [int(step_max[t]) for t in range(P)],
            "rank_total": [int(rank_total[r]) for r in range(P)]}


def pec_balance_batches(lengths, replicas):
    """Token-balanced assignment of short requests to replicas (see include/pec.h): (assign, tokens)."""
    lib = load()
    n = len(lengths)
    arr = (ctypes.c_int32 * max(n, 1))(*lengths)
    assign = (ctypes.c_int32 * max(n, 1))()
    tokens = (ctypes.c_int64 * max(replicas, 1))()
    _check(lib.pec_balance_batches(arr, n, replicas, assign, tokens))
    return [int(assign[i]) for i in range(n)], [int(tokens[r]) for r in range(replicas)]
