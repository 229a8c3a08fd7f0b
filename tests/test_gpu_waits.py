"""Bounded device-side waits: a wait that runs out is reported to the host and leaves the device usable.

The failure is made in the one form that harms nothing: a single warp waits, with the kernels' own wait routine
and a short cycle limit, on a barrier that nobody arrives on (tdq_selftest_wait_timeout).  No copy and no
tensor-core operation is in flight when it gives up, nothing traps, and the calls that follow must work."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from parity_utils import compare_y, to_cuda

pytestmark = pytest.mark.gpu


def test_linear_wait_that_runs_out_is_reported_and_the_workspace_stays_usable():
    from paper_2604_16855_b200 import tdq
    case = si.config1()
    x = case.x.reshape(-1, case.C)
    xa, wq = oracle.quantize_act(x), oracle.quantize_weight(case.w)
    ops = [to_cuda(xa["codes"]), to_cuda(xa["scale"]), to_cuda(wq["codes"]), to_cuda(wq["scale"])]
    wsp = tdq.linear_workspace(x.shape[0], case.C, case.O, 32, "cuda")
    y_before = tdq.w4a4_linear(*ops, workspace=wsp)
    assert tdq.workspace_status(wsp) == (tdq.OK, 0)
    tdq.selftest_wait_timeout(0, 300000, wsp)                 # about 0.15 ms at the SM clock
    st, detail = tdq.workspace_status(wsp)
    assert st == tdq.ERR_DEVICE_TIMEOUT
    assert detail & 0xFF == 15 and detail >> 8 == 0           # the self-test's wait, thread block 0
    assert tdq.status_string(st) == "a bounded device-side wait ran out"
    # the same workspace, the same stream: the next call clears the word and computes the same bits
    y_after = tdq.w4a4_linear(*ops, workspace=wsp)
    assert tdq.workspace_status(wsp) == (tdq.OK, 0)
    assert torch.equal(y_before.view(torch.int32), y_after.view(torch.int32))
    ref = oracle.w4a4_linear(xa["codes"], xa["scale"], wq["codes"], wq["scale"])
    compare_y(y_after.cpu().numpy(), ref, case.C // 32)


def test_quantizer_wait_that_runs_out_is_reported_once_and_the_device_stays_usable():
    from paper_2604_16855_b200 import tdq
    case = si.config2()
    x = case.x.reshape(-1, case.C)[:4096]
    xt = to_cuda(x, bf16=True)
    tdq.quantize_act(xt)
    assert tdq.quantize_status() == (tdq.OK, 0)
    tdq.selftest_wait_timeout(1, 300000)
    st, detail = tdq.quantize_status()
    assert st == tdq.ERR_DEVICE_TIMEOUT and detail & 0xFF == 14
    assert tdq.quantize_status() == (tdq.OK, 0)               # the query cleared the word
    codes, scale = tdq.quantize_act(xt)
    assert tdq.quantize_status() == (tdq.OK, 0)
    ref = oracle.quantize_act(x)
    np.testing.assert_array_equal(codes.cpu().numpy(), ref["codes"])
    np.testing.assert_array_equal(scale.cpu().numpy(), ref["scale"])
