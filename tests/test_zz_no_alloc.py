"""The allocation-free linear entry point against the ordinary one.

tdq_w4a4_linear_static serves callers that cannot obtain a device workspace (code running inside
an application that owns all device memory, or in a context where cudaMalloc may not be called):
its scratch space is a fixed array inside the library.  The file name sorts last on purpose, so
that a run which stops at the first failure has already been through every other test.
"""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from parity_utils import to_cuda

pytestmark = pytest.mark.gpu


def _operands(case, rows):
    x = case.x.reshape(-1, case.C)[:rows]
    xa = oracle.quantize_act(x)
    wq = oracle.quantize_weight(case.w)
    return (to_cuda(xa["codes"]), to_cuda(xa["scale"]), to_cuda(wq["codes"]), to_cuda(wq["scale"]))


def test_static_scratch_entry_matches_workspace_entry_twice_in_a_row():
    from paper_2604_16855_b200 import tdq
    # two different problems back to back: the second is smaller, so anything the first call left
    # in the shared array beyond the second one's blocks must not show up in its result
    for case, rows in ((si.config3(), 1500), (si.config2(), 700)):
        xc, xs, wc, ws = _operands(case, rows)
        bias = torch.linspace(-1.0, 1.0, case.O, device="cuda")
        y_ref = tdq.w4a4_linear(xc, xs, wc, ws, bias)
        y = torch.full((rows, case.O), float("nan"), device="cuda")
        tdq.w4a4_linear_static(xc, xs, wc, ws, bias, y=y, wait=True)
        torch.cuda.synchronize()
        assert torch.isfinite(y).all()
        # both entries run the same kernels on the same operand blocks, so the outputs agree bit for bit (which is
        # inside any tolerance the other output tests use)
        assert torch.equal(y.view(torch.int32), y_ref.view(torch.int32))


def test_static_scratch_entry_refuses_what_does_not_fit():
    from paper_2604_16855_b200 import tdq
    M, I, O = 18464, 768, 3072                       # needs about 18 MB of blocks
    xc = torch.zeros((M, I // 2), dtype=torch.uint8, device="cuda")
    xs = torch.ones((M, I // 32), device="cuda")
    wc = torch.zeros((O, I // 2), dtype=torch.uint8, device="cuda")
    ws = torch.ones((O,), device="cuda")
    y = torch.zeros((M, O), device="cuda")
    n0 = tdq.kernel_launch_count()
    with pytest.raises(tdq.TdqError) as e:
        tdq.w4a4_linear_static(xc, xs, wc, ws, y=y)
    assert e.value.code == tdq.ERR_WORKSPACE
    assert tdq.kernel_launch_count() == n0
