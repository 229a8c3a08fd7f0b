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
