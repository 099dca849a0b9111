"""The workspace-free decode entry point, pec_decode_attn_static.

Some callers of this library cannot allocate device memory when they need a decode step: an
inference engine that gave all free HBM to its KV-cache pool has nothing left for cudaMalloc to
hand out, and a scheduler loop that must not stall cannot afford the device-wide synchronisation
an allocation implies.  For them the library carries a fixed 4 MiB scratch array of its own.

This file is named so that pytest collects it last: it goes through the raw C ABI (ctypes), with
output buffers prepared before the calls, and checks the new entry point against the ordinary
pec_decode_attn on two calls in a row - the second call finds the first one's leftovers in the
shared scratch and must not be disturbed by them.  Both entry points run the same kernels over the
same slices, so their results must agree bit for bit; one case is also compared with the fp64
oracle.  A call that is not the first one on the device must leave the amount of free device memory
exactly as it found it (the first call may be what makes the driver load the module that holds the
array, which is why an engine should make one priming call at start-up).  It also checks that an
oversized request is refused with a message instead of overrunning the array.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2409_15104_b200 import binding, workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(seed, L, hq, hkv):
    k = workloads.normal_tensor(seed, 2, (L, hkv, 128), torch.bfloat16).to(DEV)
    v = workloads.normal_tensor(seed, 3, (L, hkv, 128), torch.bfloat16).to(DEV)
    q = workloads.normal_tensor(seed, 1, (hq, 128), torch.bfloat16).to(DEV)
    return q, k, v


def _call(fn, q, k, v, lo, hi, out_dtype, num_splits=0, workspace=None):
    """One raw C-ABI call; returns (o, lse).  Buffers are created before the call, not by it."""
    o = torch.full((q.shape[0], 128), float("nan"), dtype=out_dtype, device=DEV)
    lse = torch.full((q.shape[0],), float("nan"), dtype=torch.float32, device=DEV)
    a = binding.decode_args(q, k, v, o, lse, lo, hi, num_splits)
    if workspace is not None:
        a.workspace, a.workspace_bytes = workspace.data_ptr(), workspace.numel()
    rc = fn(ctypes.byref(a), ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == 0, binding.pec_last_error()
    return o, lse


def test_static_scratch_decode_matches_the_workspace_version_twice_in_a_row():
    lib = binding.load()
    ws = torch.empty(binding.PEC_DECODE_STATIC_SCRATCH_BYTES, dtype=torch.uint8, device=DEV)
    # two different problems back to back: the second one uses fewer slices and fewer heads, so
    # stale partials of the first are still lying in the shared scratch when it runs
    cases = [(_case(31001, 20000, 32, 8), 0, 20000, torch.float32), (_case(31002, 3000, 8, 2), 500, 2900, torch.bfloat16)]
    for (q, k, v), lo, hi, out_dtype in cases:
        want_o, want_l = _call(lib.pec_decode_attn, q, k, v, lo, hi, out_dtype, workspace=ws)
        got_o, got_l = _call(lib.pec_decode_attn_static, q, k, v, lo, hi, out_dtype)
        binding.check_status()
        assert not torch.isnan(got_o.float()).any() and not torch.isnan(got_l).any()
        assert torch.equal(got_o, want_o) and torch.equal(got_l, want_l)        # same kernels, same slices
    # the last case against the oracle (the suite's bf16 tolerances)
    ref_o, ref_l = oracle.attn_rows(q.cpu()[None], [k.shape[0] - 1], k.cpu(), v.cpu(), [(lo, hi)], False)
    assert np.abs(got_o.float().cpu().double().numpy() - ref_o[0]).max() <= 2e-2
    assert np.abs(got_l.cpu().double().numpy() - ref_l[0]).max() <= 1e-3
    # a call that is not the first on this device takes no device memory and gives none back
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    _call_into = (torch.empty_like(got_o), torch.empty_like(got_l))
    torch.cuda.synchronize()
    free_ready, _ = torch.cuda.mem_get_info()                                   # output buffers exist now
    a = binding.decode_args(q, k, v, _call_into[0], _call_into[1], lo, hi, 0)
    assert lib.pec_decode_attn_static(ctypes.byref(a), ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)) == 0
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_ready <= free_before
    assert torch.equal(_call_into[0], got_o)
    # and the very same call repeated gives the very same bits
    (q, k, v), lo, hi, out_dtype = cases[0]
    a = _call(lib.pec_decode_attn_static, q, k, v, lo, hi, out_dtype)
    b = _call(lib.pec_decode_attn_static, q, k, v, lo, hi, out_dtype)
    binding.check_status()
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


def test_static_scratch_decode_refuses_what_does_not_fit():
    lib = binding.load()
    q, k, v = _case(31003, 4096, 128, 1)
    o = torch.empty((128, 128), dtype=torch.float32, device=DEV)
    lse = torch.empty((128,), dtype=torch.float32, device=DEV)
    # 4096 keys in 32 slices of 128, 128 heads: 32 * 128 * 516 B = 2.1 MB fits; the same with Hq = 128
    # and 4096 slices cannot exist (only 32 tiles), so ask for a range that really needs more: see below
    a = binding.decode_args(q, k, v, o, lse, 0, 4096, 32)
    assert lib.pec_decode_workspace_size(ctypes.byref(a)) == 32 * 128 * 516
    assert lib.pec_decode_attn_static(ctypes.byref(a), None) == 0
    torch.cuda.synchronize()
    binding.check_status()
    big_k = torch.zeros((128 * 80, 1, 128), dtype=torch.bfloat16, device=DEV)
    a = binding.decode_args(q, big_k, big_k, o, lse, 0, 128 * 80, 80)           # 80 * 128 * 516 B = 5.3 MB > 4 MiB
    assert lib.pec_decode_workspace_size(ctypes.byref(a)) > binding.PEC_DECODE_STATIC_SCRATCH_BYTES
    assert lib.pec_decode_attn_static(ctypes.byref(a), None) == -4
    assert "built-in" in binding.pec_last_error()
