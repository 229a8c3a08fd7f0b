"""The C-ABI library loads, exports every symbol the header declares, and its host-side
argument checks answer with status codes before anything is launched (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def tdq():
    from paper_2604_16855_b200 import build
    build.build()
    from paper_2604_16855_b200 import tdq
    return tdq


def _declared():
    text = open(os.path.join(ROOT, "include", "tdq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tdq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(tdq):
    names = _declared()
    assert len(names) >= 10
    for n in names:
        assert hasattr(tdq.lib(), n), n
    assert sorted(tdq.EXPORTS) == names


def test_status_strings(tdq):
    seen = {tdq.status_string(i) for i in range(7)}
    assert len(seen) == 7 and "ok" in seen
    assert tdq.status_string(99) == "unknown status"


def test_default_params_are_the_papers(tdq):
    p = tdq.default_act_params()
    assert (p.group_size, p.tau, p.base_percentile, p.flags) == (32, 1.0, 1.0, 3)
    assert abs(p.zr - 0.2) < 1e-7


def test_bad_arguments_return_codes_without_launching(tdq):
    L = tdq.lib()
    p = tdq.default_act_params()
    fake = ctypes.c_void_p(0x1000)       # never dereferenced: every call below fails its checks first
    n0 = tdq.kernel_launch_count()
    rp = ctypes.byref(p)
    assert L.tdq_quantize_act(None, 0, 1, 4, 64, 64, rp, fake, fake, None, None) == tdq.ERR_INVALID_ARG
    assert L.tdq_quantize_act(fake, 0, 1, 4, 64, 64, None, fake, fake, None, None) == tdq.ERR_INVALID_ARG
    assert L.tdq_quantize_act(fake, 0, 1, 4, 64, 32, rp, fake, fake, None, None) == tdq.ERR_INVALID_ARG
    assert L.tdq_quantize_act(fake, 0, 1, 4, 0, 64, rp, fake, fake, None, None) == tdq.ERR_INVALID_ARG
    assert L.tdq_quantize_act(fake, 7, 1, 4, 64, 64, rp, fake, fake, None, None) == tdq.ERR_INVALID_ARG
    assert L.tdq_quantize_act(fake, 0, 1, 4, 64, 64, rp, None, fake, None, None) == tdq.ERR_INVALID_ARG
    for bad in (tdq.act_params(g=31), tdq.act_params(g=0), tdq.act_params(g=8192), tdq.act_params(tau=0.0),
                tdq.act_params(zr=0.0), tdq.act_params(zr=1.5), tdq.act_params(p=0.0), tdq.act_params(flags=8)):
        assert L.tdq_quantize_act(fake, 0, 1, 4, 64, 64, ctypes.byref(bad), fake, fake, None, None) \
            == tdq.ERR_INVALID_ARG
    assert L.tdq_quantize_act(fake, 0, 0, 4, 64, 64, rp, fake, fake, None, None) == tdq.OK      # empty: no-op
    assert L.tdq_quantize_weight(None, 0, 4, 64, 32, fake, fake, None) == tdq.ERR_INVALID_ARG
    assert L.tdq_quantize_weight(fake, 0, 4, 64, 3, fake, fake, None) == tdq.ERR_INVALID_ARG
    assert L.tdq_quantize_weight(fake, 0, 0, 64, 32, fake, fake, None) == tdq.OK
    ws = 1 << 20
    lin = lambda *a: L.tdq_w4a4_linear(*a)
    assert lin(None, fake, fake, fake, None, 4, 64, 8, 32, fake, 0, 8, None, fake, ws, None) == tdq.ERR_INVALID_ARG
    assert lin(fake, fake, fake, fake, None, 4, 64, 8, 48, fake, 0, 8, None, fake, ws, None) == tdq.ERR_INVALID_ARG
    assert lin(fake, fake, fake, fake, None, 4, 64, 8, 16, fake, 0, 8, None, fake, ws, None) == tdq.ERR_UNSUPPORTED
    assert lin(fake, fake, fake, fake, None, 4, 64, 8, 32, fake, 0, 4, None, fake, ws, None) == tdq.ERR_INVALID_ARG
    assert lin(fake, fake, fake, fake, None, 4, 64, 8, 32, fake, 0, 8, None, None, ws, None) == tdq.ERR_WORKSPACE
    assert lin(fake, fake, fake, fake, None, 4, 64, 8, 32, fake, 0, 8, None, fake, 1, None) == tdq.ERR_WORKSPACE
    odd = ctypes.c_void_p(0x1001)
    assert lin(odd, fake, fake, fake, None, 4, 64, 8, 32, fake, 0, 8, None, fake, ws, None) == tdq.ERR_ALIGNMENT
    assert lin(fake, fake, fake, fake, None, 0, 64, 8, 32, fake, 0, 8, None, fake, ws, None) == tdq.OK
    assert L.tdq_workspace_status(None, None, None) == tdq.ERR_INVALID_ARG
    assert int(L.tdq_linear_workspace_bytes(128, 64, 64, 32)) >= 16
    assert tdq.kernel_launch_count() == n0


def test_binding_refuses_cpu_tensors(tdq):
    import torch
    with pytest.raises(ValueError):
        tdq.quantize_act(torch.zeros(4, 64))


@pytest.mark.gpu
def test_binding_refuses_layouts_the_abi_cannot_see(tdq):
    """dtype, contiguity and column pitch are checked before any pointer reaches the library (no launch)."""
    import torch
    n0 = tdq.kernel_launch_count()
    xc = torch.zeros((8, 32), dtype=torch.uint8, device="cuda")
    xs = torch.ones((8, 2), device="cuda")
    wc = torch.zeros((16, 32), dtype=torch.uint8, device="cuda")
    ws = torch.ones((16,), device="cuda")
    with pytest.raises(TypeError):
        tdq.w4a4_linear(xc, xs.double(), wc, ws)
    with pytest.raises(TypeError):
        tdq.w4a4_linear(xc.to(torch.int8), xs, wc, ws)
    with pytest.raises(ValueError):
        tdq.w4a4_linear(xc, xs, wc.t().contiguous().t(), ws)                 # transposed view
    with pytest.raises(ValueError):
        tdq.w4a4_linear(xc, xs, wc, ws, y=torch.zeros((16, 8), device="cuda").t())   # columns not adjacent
    with pytest.raises(ValueError):
        tdq.w4a4_linear(xc, xs, wc, torch.ones((32,), device="cuda")[::2])
    assert tdq.kernel_launch_count() == n0


def test_wait_selftest_and_host_call_argument_checks(tdq):
    L = tdq.lib()
    fake = ctypes.c_void_p(0x1000)
    n0 = tdq.kernel_launch_count()
    assert L.tdq_selftest_wait_timeout(2, 100000, fake, None) == tdq.ERR_INVALID_ARG
    assert L.tdq_selftest_wait_timeout(0, 10, fake, None) == tdq.ERR_INVALID_ARG
    assert L.tdq_selftest_wait_timeout(0, 1 << 40, fake, None) == tdq.ERR_INVALID_ARG
    assert L.tdq_selftest_wait_timeout(0, 100000, None, None) == tdq.ERR_INVALID_ARG
    assert L.tdq_selftest_wait_timeout(0, 100000, ctypes.c_void_p(0x1004), None) == tdq.ERR_ALIGNMENT
    # the host-buffer call refuses what either of its two calls would refuse, before it queues anything
    p = tdq.default_act_params()
    host = lambda pp, ws_bytes, O=64, C=64: L.tdq_quant_linear_host(fake, 1, 1, 256, C, ctypes.byref(pp), fake, fake, None, O,
                                                                   fake, 0, fake, fake, fake, fake, fake, ws_bytes, None)
    assert host(tdq.act_params(g=16), 1 << 24) == tdq.ERR_UNSUPPORTED          # the linear layer wants g % 32 == 0
    assert host(tdq.act_params(tau=0.0), 1 << 24) == tdq.ERR_INVALID_ARG
    assert host(p, 64) == tdq.ERR_WORKSPACE
    assert host(p, 1 << 24, O=0) == tdq.ERR_INVALID_ARG
    assert tdq.kernel_launch_count() == n0
