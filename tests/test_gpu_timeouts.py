"""The bounded waits inside the tensor-core kernels: a wait that runs out must end the launch through the
kernel's normal exit with PEC_ERR_TIMEOUT in the status word, and leave the device usable.  The failure is
made by the loader leaving out one tile (a test hook behind pec_control), never by a fault: every other
wait of the CTA sees the abort flag, nothing is left spinning, tensor memory is released."""
import numpy as np
import pytest
import torch

import oracle
from helpers import TOL, compare
from paper_2409_15104_b200 import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SHORT_LIMIT = 4_000_000          # SM clock cycles: about 2 ms


@pytest.fixture
def short_waits(pec):
    """A few-millisecond wait limit and the loader hook, both restored afterwards."""
    pec.pec_control(pec.PEC_CTL_WAIT_LIMIT_CYCLES, SHORT_LIMIT)
    pec.pec_control(pec.PEC_CTL_TEST_SKIP_LAST_LOAD, 1)
    try:
        yield
    finally:
        pec.pec_control(pec.PEC_CTL_TEST_SKIP_LAST_LOAD, 0)
        pec.pec_control(pec.PEC_CTL_WAIT_LIMIT_CYCLES, 2_000_000_000)


def test_attention_wait_runs_out_and_the_next_launch_is_fine(pec, short_waits):
    S = 256                                                   # one CTA; its second stage walks two key tiles
    q, k, v = workloads.qkv(21000, S, 1, 1, 128, torch.bfloat16)
    dq, dk, dv = q.to(DEV), k.to(DEV), v.to(DEV)
    pec.check_status()
    pec.pec_prefill_attn(dq, dk, dv)                          # the last V tile never arrives
    torch.cuda.synchronize()                                  # returns: the kernel gave up by itself
    with pytest.raises(pec.PecError) as err:
        pec.check_status()
    assert err.value.code == pec.PEC_ERR_TIMEOUT
    pec.pec_control(pec.PEC_CTL_TEST_SKIP_LAST_LOAD, 0)
    o, lse = pec.pec_prefill_attn(dq, dk, dv)                 # same device, same context, still the short limit
    pec.check_status()
    compare(o, lse, *oracle.prefill_attn(q, k, v, seq_len=S), *TOL[torch.bfloat16], "launch after a timeout")


def test_linear_pair_leaves_together_when_a_wait_runs_out(pec, short_waits):
    M, N, K = 256, 256, 128                                   # one CTA pair, two K steps
    x = workloads.normal_tensor(21001, 1, (M, K), torch.bfloat16)
    w = (workloads.normal_tensor(21002, 2, (N, K), torch.float32) / K ** 0.5).to(torch.bfloat16)
    dx, dw = x.to(DEV), w.to(DEV)
    pec.check_status()
    pec.pec_linear(dx, dw)                                    # the second CTA's last K step never arrives
    torch.cuda.synchronize()
    with pytest.raises(pec.PecError) as err:
        pec.check_status()
    assert err.value.code == pec.PEC_ERR_TIMEOUT
    pec.pec_control(pec.PEC_CTL_TEST_SKIP_LAST_LOAD, 0)
    y = pec.pec_linear(dx, dw)
    pec.check_status()
    assert np.abs(y.float().cpu().double().numpy() - oracle.linear(x, w)).max() <= 2e-2


def test_linear_merged_pair_leaves_together_when_a_wait_runs_out(pec, short_waits):
    rows, hq, N = 256, 1, 512                                 # one CTA pair, two K steps
    os_ = [workloads.normal_tensor(21010 + i, 1, (rows, hq, 128), torch.float32) for i in range(2)]
    ls_ = [workloads.normal_tensor(21020 + i, 2, (rows, hq), torch.float32) for i in range(2)]
    w = (workloads.normal_tensor(21003, 3, (N, hq * 128), torch.float32) / 128 ** 0.5).to(torch.bfloat16)
    do, dl, dw = [o.to(DEV) for o in os_], [l.to(DEV) for l in ls_], w.to(DEV)
    pec.check_status()
    pec.pec_linear_merged(do, dl, dw)                         # the second CTA's last K step of w never arrives
    torch.cuda.synchronize()
    with pytest.raises(pec.PecError) as err:
        pec.check_status()
    assert err.value.code == pec.PEC_ERR_TIMEOUT
    pec.pec_control(pec.PEC_CTL_TEST_SKIP_LAST_LOAD, 0)
    y = pec.pec_linear_merged(do, dl, dw)
    pec.check_status()
    merged, _ = oracle.merge_n([o.numpy() for o in os_], [l.numpy() for l in ls_])
    want = oracle.linear(torch.from_numpy(merged.reshape(rows, hq * 128)), w)
    assert np.abs(y.float().cpu().double().numpy() - want).max() <= 2e-2


def test_control_rejects_unknown_settings(pec):
    with pytest.raises(pec.PecError):
        pec.pec_control(99, 1)
    with pytest.raises(pec.PecError):
        pec.pec_control(pec.PEC_CTL_WAIT_LIMIT_CYCLES, 5)
    with pytest.raises(pec.PecError):
        pec.pec_control(pec.PEC_CTL_TEST_SKIP_LAST_LOAD, 2)
