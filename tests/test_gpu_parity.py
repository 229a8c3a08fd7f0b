"""GPU parity: every C-ABI entry point against the CPU oracle on the same seeded inputs.
All tests call through the ctypes binding of libtdq.so; the rules are in parity_utils."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from parity_utils import case_tensors, compare_quantizer, compare_y, to_cuda, unpack_codes

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tdq():
    from paper_2604_16855_b200 import tdq
    return tdq


def _quant_both(tdq, x_np, bf16, **kw):
    """(oracle dict, gpu codes, gpu scale) for x_np [M, C] (float32, or uint16 bf16 bits)."""
    g = kw.get("g", 32)
    ref = oracle.quantize_act(x_np, **kw)
    params = tdq.act_params(g=g, tau=kw.get("tau", 1.0), zr=kw.get("zr", 0.2), p=kw.get("p", 1.0),
                            flags=kw.get("flags", 3))
    codes, scale = tdq.quantize_act(to_cuda(x_np, bf16=bf16), params)
    torch.cuda.synchronize()
    return ref, codes.cpu().numpy(), scale.cpu().numpy()


def _f32(x_np, bf16):
    return si.bf16_bits_to_f32(x_np) if bf16 else x_np


# ---------------------------------------------------------------------------------------
# quantizer

@pytest.mark.parametrize("idx", [1, 2, 3, 4])
def test_quantizer_matches_oracle_on_workloads(tdq, idx):
    case = si.config(idx)
    x = case.x.reshape(-1, case.C)
    ref, codes, scale = _quant_both(tdq, x, case.x_is_bf16)
    rep = compare_quantizer(_f32(x, case.x_is_bf16), 32, ref, codes, scale)
    print("cfg%d quantizer parity: %s" % (idx, rep))
    assert rep["scale_exact_frac"] == 1.0


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("tau,zr,flags", [(1.0, 0.2, 3), (0.5, 0.2, 3), (0.25, 0.1, 3), (1.0, 0.5, 3),
                                          (1.0, 0.2, 1), (1.0, 0.2, 2), (1.0, 0.2, 0), (0.3, 0.4, 3), (2.0, 1.0, 3), (1.0, 0.3, 3), (0.7, 1.0, 2)])
def test_quantizer_fast_path_settings_and_c1_binding(tdq, bf16, tau, zr, flags):
    xs = [si.dc_offset_tokens(M=700, C=96), si.config1().x.reshape(-1, 64), si.edge_rows(C=64)]
    for x in xs:
        if bf16:
            x = si.f32_to_bf16_bits(x)
        ref, codes, scale = _quant_both(tdq, x, bf16, tau=tau, zr=zr, flags=flags)
        rep = compare_quantizer(_f32(x, bf16), 32, ref, codes, scale)
        assert rep["scale_exact_frac"] == 1.0, rep


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("C,g", [(48, 32), (72, 32), (100, 32), (64, 16), (128, 64), (96, 96), (320, 320),
                                 (70, 14), (4096, 4096), (30, 32)])
def test_quantizer_generic_path_padding_and_group_sizes(tdq, bf16, C, g):
    rng = np.random.default_rng(C * 1000 + g)
    x = si.token_mixture(rng, 1, 37, C, sigma_log_std=0.5, bg_frac=0.1, bg_nu=3.0, bg_amp=20.0).reshape(-1, C)
    x[::5] += 2.0                                    # some C1-bound groups
    if bf16:
        x = si.f32_to_bf16_bits(x)
    for kw in (dict(), dict(p=0.9), dict(tau=0.5, zr=0.3)):
        ref, codes, scale = _quant_both(tdq, x, bf16, g=g, **kw)
        rep = compare_quantizer(_f32(x, bf16), g, ref, codes, scale)
        assert rep["scale_max_rel"] <= 1e-6


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("rank", [1, 2, 3, 5, 6, 8, 9, 11, 12, 14, 15, 17, 18, 21, 24, 27, 28, 30, 31])
def test_quantizer_every_zero_bin_rank_on_the_fast_path(tdq, bf16, rank):
    # zr chosen so that ceil(zr * 32) is the rank; the ranks of the other fast-path tests are left out
    zr = (rank - 0.5) / 32.0
    xs = [si.dc_offset_tokens(M=300, C=96), si.config1().x.reshape(-1, 64), si.edge_rows(C=64)]
    for x in xs:
        if bf16:
            x = si.f32_to_bf16_bits(x)
        ref, codes, scale = _quant_both(tdq, x, bf16, zr=zr)
        rep = compare_quantizer(_f32(x, bf16), 32, ref, codes, scale)
        assert rep["scale_exact_frac"] == 1.0, rep


def test_quantizer_percentile_and_odd_rank_settings(tdq):
    x = si.config1().x.reshape(-1, 64)
    for kw in (dict(p=0.9), dict(zr=0.27), dict(zr=0.95, p=0.5)):
        ref, codes, scale = _quant_both(tdq, x, False, **kw)
        compare_quantizer(x, 32, ref, codes, scale)


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("p,flags", [(0.9, 3), (0.92, 3), (0.95, 3), (0.9, 1), (0.95, 0), (0.92, 2)])
def test_quantizer_percentile_base_radius_on_the_fast_path(tdq, bf16, p, flags):
    # ranks 29, 30 and 31 of 32 (Supp. S4.8's percentile option) on dense rows and on rows with a pitch
    xs = [si.dc_offset_tokens(M=700, C=96), si.config1().x.reshape(-1, 64), si.edge_rows(C=64)]
    for x in xs:
        if bf16:
            x = si.f32_to_bf16_bits(x)
        ref, codes, scale = _quant_both(tdq, x, bf16, p=p, flags=flags)
        rep = compare_quantizer(_f32(x, bf16), 32, ref, codes, scale)
        assert rep["scale_exact_frac"] == 1.0, rep
        wide = np.zeros((x.shape[0], x.shape[1] + 32), x.dtype)
        wide[:, : x.shape[1]] = x
        xt = to_cuda(wide, bf16=bf16)[:, : x.shape[1]]
        c2, s2 = tdq.quantize_act(xt, tdq.act_params(p=p, flags=flags))
        np.testing.assert_array_equal(c2.cpu().numpy(), codes)
        np.testing.assert_array_equal(s2.cpu().numpy(), scale)


def test_quantizer_row_stride_offset_output_and_empty(tdq):
    case = si.config2()
    bits = case.x.reshape(-1, 64)[:1000]
    wide = np.full((1000, 96), 0x7F7F, np.uint16)
    wide[:, :64] = bits
    xt = to_cuda(wide, bf16=True)[:, :64]            # row stride 96 elements, fast path
    ref = oracle.quantize_act(bits)
    off = torch.full((1000, 2), 5.0, device="cuda")
    codes, scale = tdq.quantize_act(xt, offset=off)
    compare_quantizer(si.bf16_bits_to_f32(bits), 32, ref, codes.cpu().numpy(), scale.cpu().numpy())
    assert (off == 0).all()
    wide2 = np.full((1000, 75), 0x7F7F, np.uint16)   # stride 75: unaligned rows -> generic kernel
    wide2[:, :64] = bits
    codes, scale = tdq.quantize_act(to_cuda(wide2, bf16=True)[:, :64])
    compare_quantizer(si.bf16_bits_to_f32(bits), 32, ref, codes.cpu().numpy(), scale.cpu().numpy())
    c0, s0 = tdq.quantize_act(torch.empty((0, 64), device="cuda"))
    assert c0.shape == (0, 32) and s0.shape == (0, 2)


def test_quantizer_does_not_write_outside_its_outputs(tdq):
    x = to_cuda(si.config1().x.reshape(-1, 64)[:77])
    codes = torch.full((77 * 32 + 64,), 0xAB, dtype=torch.uint8, device="cuda")
    scale = torch.full((77 * 2 + 16,), -1.0, device="cuda")
    tdq.quantize_act(x, codes=codes[32:32 + 77 * 32].view(77, 32), scale=scale[8:8 + 154].view(77, 2))
    torch.cuda.synchronize()
    assert (codes[:32] == 0xAB).all() and (codes[-32:] == 0xAB).all()
    assert (scale[:8] == -1).all() and (scale[-8:] == -1).all()


# ---------------------------------------------------------------------------------------
# weight quantizer

@pytest.mark.parametrize("O,I,bf16", [(64, 64, False), (256, 64, False), (40, 100, False), (960, 320, True), (3, 7, False)])
def test_weight_quantizer_matches_oracle(tdq, O, I, bf16):
    rng = np.random.default_rng(O + I)
    w = si.weights(rng, O, I)
    w[0] = 0.0
    w_np = si.f32_to_bf16_bits(w) if bf16 else w
    ref = oracle.quantize_weight(w_np, pad_to=32)
    wc, ws = tdq.quantize_weight(to_cuda(w_np, bf16=bf16), 32)
    np.testing.assert_array_equal(ws.cpu().numpy(), ref["scale"])
    np.testing.assert_array_equal(wc.cpu().numpy(), ref["codes"])


# ---------------------------------------------------------------------------------------
# linear layer

def _linear_case(tdq, x_np, bf16, w_np, g=32, bias=None, out_dtype=torch.float32, want_acc=True, rows=None, **kw):
    xa = oracle.quantize_act(x_np, g=g, **kw)
    wq = oracle.quantize_weight(w_np, pad_to=g)
    xc, xs = to_cuda(xa["codes"]), to_cuda(xa["scale"])
    wc, ws = to_cuda(wq["codes"]), to_cuda(wq["scale"])
    M, O, K = xa["codes"].shape[0], w_np.shape[0], xa["scale"].shape[1]
    acc = torch.full((M, O, K), 12345, dtype=torch.int32, device="cuda") if want_acc else None
    b = None if bias is None else to_cuda(bias)
    wsp = tdq.linear_workspace(M, K * g, O, g, "cuda")
    y = tdq.w4a4_linear(xc, xs, wc, ws, b, g=g, out_dtype=out_dtype, acc_debug=acc, workspace=wsp)
    st, detail = tdq.workspace_status(wsp)
    assert st == tdq.OK, "device wait ran out: 0x%x" % detail
    sel = slice(None) if rows is None else rows
    ref = oracle.w4a4_linear(xa["codes"][sel], xa["scale"][sel], wq["codes"], wq["scale"], bias=bias, g=g,
                             want_acc=want_acc)
    if want_acc:
        np.testing.assert_array_equal(acc.cpu().numpy()[sel], ref["acc"])     # bit-exact integer sums
    return y.float().cpu().numpy()[sel], ref


@pytest.mark.parametrize("idx", [1, 2])
def test_linear_matches_oracle_small_workloads(tdq, idx):
    case = si.config(idx)
    x = case.x.reshape(-1, case.C)
    if idx == 2:
        x = x[:3000]
    y, ref = _linear_case(tdq, x, case.x_is_bf16, case.w)
    worst, strict = compare_y(y, ref, 2)
    print("cfg%d linear: worst err/tol %.3f, %.6f of outputs within 1e-5 relative" % (idx, worst, strict))
    assert strict > 0.99


@pytest.mark.parametrize("M,C,O,g", [(1, 32, 8, 32), (129, 64, 65, 32), (300, 96, 200, 32), (257, 320, 130, 32),
                                     (100, 128, 64, 64), (130, 256, 96, 128), (64, 768, 72, 768), (50, 100, 30, 32),
                                     # more work items than SMs: a CTA takes several row blocks in turn
                                     (19200, 32, 128, 32), (2100, 64, 1280, 32), (19100, 64, 100, 64)])
def test_linear_shapes_tails_bias_and_wide_groups(tdq, M, C, O, g):
    rng = np.random.default_rng(M + C + O)
    x = si.token_mixture(rng, 1, M, C, sigma_log_std=0.5, bg_frac=0.1, bg_nu=3.0, bg_amp=20.0).reshape(-1, C)
    w = si.weights(rng, O, C)
    bias = rng.standard_normal(O).astype(np.float32)
    y, ref = _linear_case(tdq, x, False, w, g=g, bias=bias)
    compare_y(y, ref, -(-C // g) + 1)


def test_linear_bf16_output_and_row_stride(tdq):
    case = si.config1()
    x = case.x.reshape(-1, 64)
    y, ref = _linear_case(tdq, x, False, case.w, out_dtype=torch.bfloat16, want_acc=False)
    compare_y(y, ref, 2, out_eps=2.0 ** -8)                         # plus one bf16 rounding
    xa = oracle.quantize_act(x)
    wq = oracle.quantize_weight(case.w)
    ybig = torch.full((256, 80), 7.0, device="cuda")
    tdq.w4a4_linear(to_cuda(xa["codes"]), to_cuda(xa["scale"]), to_cuda(wq["codes"]), to_cuda(wq["scale"]),
                    y=ybig[:, :64])
    torch.cuda.synchronize()
    compare_y(ybig[:, :64].cpu().numpy(), ref, 2)
    assert (ybig[:, 64:] == 7.0).all()


@pytest.mark.parametrize("idx", [3, 4])
def test_linear_full_size_workloads_on_sampled_rows(tdq, idx):
    case = si.config(idx)
    x = case.x.reshape(-1, case.C)
    rng = np.random.default_rng(idx)
    rows = np.sort(np.concatenate([rng.choice(x.shape[0], 160, replace=False), [0, 127, 128, x.shape[0] - 1]]))
    rows = np.unique(rows)
    y, ref = _linear_case(tdq, x, case.x_is_bf16, case.w, want_acc=False, rows=rows)
    worst, strict = compare_y(y, ref, case.C // 32)
    print("cfg%d linear (sampled %d rows): worst err/tol %.3f, %.6f within 1e-5 relative"
          % (idx, len(rows), worst, strict))
    assert strict > 0.99


def test_quantize_then_linear_end_to_end_matches_oracle(tdq):
    case = si.config3()
    x = case.x.reshape(-1, case.C)[:1500]
    xt = to_cuda(x, bf16=True)
    wc, ws = tdq.quantize_weight(to_cuda(case.w))
    codes, scale = tdq.quantize_act(xt)
    y = tdq.w4a4_linear(codes, scale, wc, ws)
    xa = oracle.quantize_act(x)
    wq = oracle.quantize_weight(case.w)
    ref = oracle.w4a4_linear(xa["codes"], xa["scale"], wq["codes"], wq["scale"])
    np.testing.assert_array_equal(codes.cpu().numpy(), xa["codes"])
    compare_y(y.cpu().numpy(), ref, case.C // 32)


def test_sweep_layers_spot_check(tdq):
    for li in (3, 11, 19, 31):                   # fc2 of each stage: the widest contraction of the stage
        case = si.config5_layer(li, batch=1)
        x = case.x.reshape(-1, case.C)[:512]
        y, ref = _linear_case(tdq, x, True, case.w, want_acc=False)
        compare_y(y, ref, case.C // 32)


# ------------------------------------------------------------------------------------------
# fused variant: the quantizer as the producer of the linear layer's A operand

@pytest.mark.gpu
@pytest.mark.parametrize("idx,rows,bf16_x,out_dtype,use_bias", [
    (1, None, False, torch.float32, False),     # cfg1: fp32 activations, two groups per row
    (2, 3000, True, torch.float32, True),       # cfg2: several row blocks per CTA, ragged last block
    (3, 1500, True, torch.float32, False),      # cfg3: ten groups per row (a ragged last quad)
    (3, 700, True, torch.bfloat16, True),
    (4, 400, True, torch.float32, False),       # cfg4: the widest contraction that stays resident
])
def test_fused_matches_oracle_and_the_two_call_path(tdq, idx, rows, bf16_x, out_dtype, use_bias):
    case = getattr(si, "config%d" % idx)()
    x = case.x.reshape(-1, case.C)
    if rows:
        x = x[:rows]
    xt = to_cuda(x, bf16=bf16_x)
    wc, ws = tdq.quantize_weight(to_cuda(case.w))
    bias_np = (np.linspace(-1.0, 1.0, case.O).astype(np.float32) * 0.01) if use_bias else None
    bias = torch.from_numpy(bias_np).cuda() if use_bias else None
    y = tdq.quant_linear_fused(xt, wc, ws, bias, out_dtype=out_dtype)
    codes, scale = tdq.quantize_act(xt)
    y2 = tdq.w4a4_linear(codes, scale, wc, ws, bias, out_dtype=out_dtype)
    # the same kernel consumes the same operand bytes and scales: bit-identical results
    assert torch.equal(y.view(torch.int16 if out_dtype == torch.bfloat16 else torch.int32),
                       y2.view(torch.int16 if out_dtype == torch.bfloat16 else torch.int32))
    if out_dtype == torch.float32:
        xa = oracle.quantize_act(_f32(x, bf16_x))
        wq = oracle.quantize_weight(case.w)
        ref = oracle.w4a4_linear(xa["codes"], xa["scale"], wq["codes"], wq["scale"], bias=bias_np)
        compare_y(y.cpu().numpy(), ref, case.C // 32)


@pytest.mark.gpu
def test_fused_settings_and_refusals(tdq):
    case = si.config3()
    x = case.x.reshape(-1, case.C)[:300]
    xt = to_cuda(x, bf16=True)
    wc, ws = tdq.quantize_weight(to_cuda(case.w))
    # C1 binding (small tau), C2 off, both off: the producer follows the same flags as the quantizer
    for tau, flags in [(0.25, 3), (1.0, 1), (1.0, 0)]:
        p = tdq.act_params(tau=tau, flags=flags)
        y = tdq.quant_linear_fused(xt, wc, ws, params=p)
        codes, scale = tdq.quantize_act(xt, p)
        y2 = tdq.w4a4_linear(codes, scale, wc, ws)
        assert torch.equal(y.view(torch.int32), y2.view(torch.int32))
    # refused: another zero-bin rank, another group size, a contraction too wide to stay in shared memory
    with pytest.raises(tdq.TdqError) as e:
        tdq.quant_linear_fused(xt, wc, ws, params=tdq.act_params(zr=0.5))
    assert e.value.code == tdq.ERR_UNSUPPORTED
    with pytest.raises(tdq.TdqError) as e:
        tdq.quant_linear_fused(xt, wc, ws, params=tdq.act_params(g=64))
    assert e.value.code == tdq.ERR_UNSUPPORTED
    with pytest.raises(tdq.TdqError) as e:          # a percentile base radius: the two-call path has it
        tdq.quant_linear_fused(xt, wc, ws, params=tdq.act_params(p=0.95))
    assert e.value.code == tdq.ERR_UNSUPPORTED
    wide = torch.zeros((64, 2048), dtype=torch.bfloat16, device="cuda")
    wcw, wsw = tdq.quantize_weight(torch.zeros((32, 2048), device="cuda"))
    with pytest.raises(tdq.TdqError) as e:
        tdq.quant_linear_fused(wide, wcw, wsw)
    assert e.value.code == tdq.ERR_UNSUPPORTED


# ------------------------------------------------------------------------------------------
# channel-major input (feature maps quantized along C in place)

def _feature_map(seed, B, C, H, W, bf16):
    rng = np.random.RandomState(seed)
    sig = np.exp(rng.normal(0.0, 0.7, size=(B, 1, H, W)))
    x = (rng.normal(size=(B, C, H, W)) * sig).astype(np.float32)
    x[rng.rand(B, C, H, W) < 0.02] *= 30.0          # a few outliers
    x[:, :, 0, 0] = 0.0                              # an all-zero token
    return si.f32_to_bf16_bits(x) if bf16 else x


@pytest.mark.gpu
@pytest.mark.parametrize("B,C,H,W,bf16", [
    (2, 64, 9, 16, True),      # 288-byte channel rows: vector loads, one tile with a tail
    (3, 32, 20, 20, True),     # 400 positions: two tiles, the second ragged
    (1, 96, 7, 9, False),      # 252-byte rows: element-wise loads
    (2, 64, 8, 8, False),      # fp32 vector loads
    (1, 320, 5, 13, True),     # 130-byte rows: element-wise loads, ten groups
])
def test_quantizer_channel_major_matches_oracle_and_the_row_major_path(tdq, B, C, H, W, bf16):
    x = _feature_map(B * 1000 + C + H, B, C, H, W, bf16)
    ref = oracle.quantize_act_nchw(x)
    xt = to_cuda(x, bf16=bf16)
    codes, scale = tdq.quantize_act_nchw(xt)
    rows = xt.permute(0, 2, 3, 1).contiguous().view(B * H * W, C)
    codes2, scale2 = tdq.quantize_act(rows)
    assert torch.equal(codes, codes2) and torch.equal(scale.view(torch.int32), scale2.view(torch.int32))
    x_tok = np.ascontiguousarray(np.transpose(x, (0, 2, 3, 1))).reshape(B * H * W, C)
    compare_quantizer(_f32(x_tok, bf16), 32, ref, codes.cpu().numpy(), scale.cpu().numpy())


@pytest.mark.gpu
def test_quantizer_channel_major_settings_and_refusals(tdq):
    x = _feature_map(7, 2, 64, 6, 8, True)
    xt = to_cuda(x, bf16=True)
    for tau, zr, flags in [(0.25, 0.2, 3), (1.0, 0.5, 3), (1.0, 0.2, 1), (1.0, 0.2, 0)]:
        p = tdq.act_params(tau=tau, zr=zr, flags=flags)
        ref = oracle.quantize_act_nchw(x, tau=tau, zr=zr, flags=flags)
        codes, scale = tdq.quantize_act_nchw(xt, p)
        np.testing.assert_array_equal(codes.cpu().numpy(), ref["codes"])
        np.testing.assert_array_equal(scale.cpu().numpy(), ref["scale"])
    for bad in (tdq.act_params(g=64), tdq.act_params(p=0.9), tdq.act_params(zr=0.25)):   # rank 8 has no fast kernel
        with pytest.raises(tdq.TdqError) as e:
            tdq.quantize_act_nchw(xt, bad)
        assert e.value.code == tdq.ERR_UNSUPPORTED
    # offsets are written when asked for, and an empty map is a no-op
    off = torch.full((2 * 48, 2), 5.0, device="cuda")
    tdq.quantize_act_nchw(xt, offset=off)
    assert float(off.abs().max()) == 0.0
    tdq.quantize_act_nchw(torch.empty((0, 64, 6, 8), dtype=torch.bfloat16, device="cuda"))


# ------------------------------------------------------------------------------------------
# fixed-radius control

@pytest.mark.gpu
@pytest.mark.parametrize("idx,bf16,g,radius", [(1, False, 32, 1.0), (2, True, 32, 0.37), (3, True, 64, 3.0),
                                               (3, True, 320, 0.05), (2, True, 8, 1e-9), (1, False, 32, 1e38)])
def test_fixed_radius_quantizer_matches_oracle(tdq, idx, bf16, g, radius):
    case = si.config(idx)
    x = case.x.reshape(-1, case.C)[:3000]
    ref = oracle.quantize_act_fixed(x, radius, g=g)
    codes, scale = tdq.quantize_act_fixed(to_cuda(x, bf16=bf16), radius, g)
    np.testing.assert_array_equal(codes.cpu().numpy(), ref["codes"])
    np.testing.assert_array_equal(scale.cpu().numpy(), ref["scale"])


@pytest.mark.gpu
def test_fixed_radius_quantizer_stride_offset_linear_and_refusals(tdq):
    case = si.config3()
    x = case.x.reshape(-1, case.C)[:520]
    wide = np.zeros((520, case.C + 24), np.uint16)
    wide[:, :case.C] = x
    xt = to_cuda(wide, bf16=True)[:, :case.C]                 # rows 344 elements apart
    off = torch.full((520, case.C // 32), 3.0, device="cuda")
    codes, scale = tdq.quantize_act_fixed(xt, 2.0, 32, offset=off)
    ref = oracle.quantize_act_fixed(x, 2.0, g=32)
    np.testing.assert_array_equal(codes.cpu().numpy(), ref["codes"])
    assert float(off.abs().max()) == 0.0
    # the outputs feed the linear layer unchanged
    wc, ws = tdq.quantize_weight(to_cuda(case.w))
    y = tdq.w4a4_linear(codes, scale, wc, ws)
    wq = oracle.quantize_weight(case.w)
    compare_y(y.cpu().numpy(), oracle.w4a4_linear(ref["codes"], ref["scale"], wq["codes"], wq["scale"]), case.C // 32)
    for g, radius, code in [(12, 1.0, tdq.ERR_UNSUPPORTED), (32, 0.0, tdq.ERR_INVALID_ARG), (96, 1.0, tdq.ERR_UNSUPPORTED)]:
        with pytest.raises(tdq.TdqError) as e:
            tdq.quantize_act_fixed(xt, radius, g)
        assert e.value.code == code


# ------------------------------------------------------------------------------------------
# power-of-two step variant

@pytest.mark.gpu
@pytest.mark.parametrize("idx,bf16,g", [(1, False, 32), (2, True, 32), (3, True, 32), (3, True, 64), (2, True, 16)])
def test_power_of_two_steps_match_oracle(tdq, idx, bf16, g):
    case = si.config(idx)
    x = case.x.reshape(-1, case.C)[:2500]
    flags = 7
    ref, codes, scale = _quant_both(tdq, x, bf16, g=g, flags=flags)
    np.testing.assert_array_equal(codes, ref["codes"])
    np.testing.assert_array_equal(scale, ref["scale"])
    assert np.all(np.frexp(scale.astype(np.float64))[0] == 0.5)


def _pow2_case(tdq, x_np, bf16, w_np, g=32, bias=None, out_dtype=torch.float32):
    xa = oracle.quantize_act(x_np, g=g, flags=7)
    wq = oracle.quantize_weight(w_np, pad_to=g)
    wsp = tdq.linear_workspace(xa["codes"].shape[0], xa["codes"].shape[1] * 2, w_np.shape[0], g, "cuda")
    y = tdq.w4a4_linear_pow2(to_cuda(xa["codes"]), to_cuda(xa["scale"]), to_cuda(wq["codes"]), to_cuda(wq["scale"]),
                             None if bias is None else to_cuda(bias), g=g, out_dtype=out_dtype, workspace=wsp)
    st, detail = tdq.workspace_status(wsp)
    assert st == tdq.OK, "status 0x%x" % detail
    ref = oracle.w4a4_linear(xa["codes"], xa["scale"], wq["codes"], wq["scale"], bias=bias, g=g)
    return y.float().cpu().numpy(), ref, xa


@pytest.mark.gpu
@pytest.mark.parametrize("idx,rows,g", [(1, None, 32), (2, 3000, 32), (3, 1500, 32), (3, 700, 64), (4, 300, 32)])
def test_power_of_two_linear_matches_the_exact_layer(tdq, idx, rows, g):
    case = si.config(idx)
    x = case.x.reshape(-1, case.C)
    if rows:
        x = x[:rows]
    bias = np.linspace(-0.02, 0.02, case.O).astype(np.float32) if idx == 3 else None
    y, ref, xa = _pow2_case(tdq, x, case.x_is_bf16, case.w, g=g, bias=bias)
    # the steps of a row span fewer than 15 binades here, so nothing is truncated; what remains is the
    # binary32 accumulation of C products in the tensor core's order
    spread = np.log2(xa["scale"].max(axis=1) / xa["scale"].min(axis=1)).max()
    assert spread <= 14
    worst, strict = compare_y(y, ref, case.C)
    assert strict > 0.99


@pytest.mark.gpu
def test_power_of_two_linear_truncation_bound_bf16_output_and_bad_scales(tdq):
    rng = np.random.RandomState(9)
    M, C, O = 200, 128, 96
    x = rng.normal(size=(M, C)).astype(np.float32)
    x[:, 32:64] *= 1e-6                                    # one group 2^20 below the others: truncated
    w = (rng.normal(size=(O, C)) * 0.02).astype(np.float32)
    y, ref, xa = _pow2_case(tdq, x, False, w)
    wq = oracle.quantize_weight(w)
    big = xa["scale"].max(axis=1, keepdims=True).astype(np.float64)
    bound = 32 * 8 * wq["scale"].astype(np.float64)[None, :] * big * 2.0 ** -14      # 32 truncated elements, |q_w| <= 8
    tol = np.maximum(1e-5 * np.abs(ref["y_d"]), (C + 2) * 2.0 ** -24 * ref["t_abs"]) + bound
    assert np.all(np.abs(y - ref["y_d"]) <= tol)
    # bf16 output and a ragged shape
    yb, refb, _ = _pow2_case(tdq, x[:131], False, w[:70], out_dtype=torch.bfloat16)
    assert np.all(np.abs(yb - refb["y_d"]) <= 2.0 ** -8 * np.abs(refb["y_d"]) + bound[:131, :70] + 1e-6)
    # a step that is not a power of two is reported
    xa2 = oracle.quantize_act(x)                           # the paper's steps
    wsp = tdq.linear_workspace(M, C, O, 32, "cuda")
    tdq.w4a4_linear_pow2(to_cuda(xa2["codes"]), to_cuda(xa2["scale"]), to_cuda(wq["codes"]), to_cuda(wq["scale"]), workspace=wsp)
    st, detail = tdq.workspace_status(wsp)
    assert st != tdq.OK and (detail & 0xff) == 11


@pytest.mark.gpu
def test_power_of_two_bad_step_report_belongs_to_its_call(tdq):
    # the report of a step that is not a power of two does not outlive its call: neither with one workspace
    # used by call after call, nor when the calls are replays of one captured graph over changing scales
    rng = np.random.RandomState(12)
    M, C, O = 300, 256, 100
    x = rng.normal(size=(M, C)).astype(np.float32)
    w = (rng.normal(size=(O, C)) * 0.02).astype(np.float32)
    good, bad = oracle.quantize_act(x, flags=7), oracle.quantize_act(x)
    wq = oracle.quantize_weight(w)
    codes, wc, ws = to_cuda(good["codes"]), to_cuda(wq["codes"]), to_cuda(wq["scale"])
    s_good, s_bad = to_cuda(good["scale"]), to_cuda(bad["scale"])
    wsp = torch.empty_like(tdq.linear_workspace(M, C, O, 32, "cuda")).fill_(0x5a)   # nothing relies on a cleared workspace
    y = torch.empty((M, O), device="cuda")
    scale = s_good.clone()

    def status():
        st, detail = tdq.workspace_status(wsp)
        return 0 if st == tdq.OK else detail & 0xff

    for want, src in [(0, s_good), (11, s_bad), (11, s_bad), (0, s_good), (0, s_good), (11, s_bad), (0, s_good)]:
        scale.copy_(src)
        tdq.w4a4_linear_pow2(codes, scale, wc, ws, y=y, workspace=wsp)
        assert status() == want
    y_good = y.clone()
    # an exact-step call in between leaves nothing behind either
    scale.copy_(s_bad)
    tdq.w4a4_linear_pow2(codes, scale, wc, ws, y=y, workspace=wsp)
    tdq.w4a4_linear(codes, scale, wc, ws, y=y, workspace=wsp)
    assert status() == 0
    tdq.w4a4_linear_pow2(codes, s_good, wc, ws, y=y, workspace=wsp)
    assert status() == 0
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        tdq.w4a4_linear_pow2(codes, scale, wc, ws, y=y, workspace=wsp)
    for want, src in [(11, s_bad), (0, s_good), (0, s_good), (11, s_bad), (11, s_bad), (0, s_good)]:
        scale.copy_(src)
        graph.replay()
        assert status() == want
    assert torch.equal(y.view(torch.int32), y_good.view(torch.int32))


# ------------------------------------------------------------------------------------------
# host-buffer entry point (chunked copies overlapped with the kernels)

@pytest.mark.gpu
@pytest.mark.parametrize("idx,rows", [(3, None), (2, 300), (1, None)])
def test_host_buffer_call_equals_the_two_calls(tdq, idx, rows):
    case = si.config(idx)
    x = case.x.reshape(-1, case.C)
    if rows:
        x = x[:rows]
    xt = to_cuda(x, bf16=case.x_is_bf16)
    wc, ws = tdq.quantize_weight(to_cuda(case.w))
    codes, scale = tdq.quantize_act(xt)
    y_ref = tdq.w4a4_linear(codes, scale, wc, ws).cpu()
    x_host = xt.cpu().pin_memory()
    for _ in range(2):                       # twice: the side streams and events are reused
        y_host, keep = tdq.quant_linear_host(x_host, wc, ws)
        torch.cuda.current_stream().synchronize()
        assert torch.equal(y_host.view(torch.int32), y_ref.view(torch.int32))
        st, detail = tdq.workspace_status(keep[0])
        assert st == tdq.OK


# ------------------------------------------------------------------------------------------
# seeded random shapes: every mode of the linear kernel (resident and streamed operands, several work
# items per CTA, one to four item buffers, in-kernel unpacking, both strip layouts) on ragged sizes

def _random_linear_shapes(n, seed=2024):
    rng = np.random.RandomState(seed)
    shapes = []
    for _ in range(n):
        C = int(rng.choice([32, 64, 96, 128, 256, 320, 512, 768, 832, 1024]))
        gs = [g for g in (32, 64, 128, C) if C % g == 0]
        g = int(gs[rng.randint(len(gs))])
        M = int(rng.choice([1, 37, 128, 129, 300, 700, 1500]))
        O = int(rng.choice([1, 8, 100, 128, 130, 384, 700]))
        shapes.append((M, C, O, g, bool(rng.randint(2)), bool(rng.randint(2))))
    return shapes


@pytest.mark.gpu
@pytest.mark.parametrize("M,C,O,g,bf16_out,with_bias", _random_linear_shapes(40))
def test_linear_random_shapes(tdq, M, C, O, g, bf16_out, with_bias):
    rng = np.random.RandomState(M * 7 + C + O)
    x = (rng.normal(size=(M, C)) * np.exp(rng.normal(0, 1.0, size=(M, 1)))).astype(np.float32)
    w = (rng.normal(size=(O, C)) * 0.05).astype(np.float32)
    bias = rng.normal(size=(O,)).astype(np.float32) * 0.1 if with_bias else None
    y, ref = _linear_case(tdq, x, False, w, g=g, bias=bias, out_dtype=torch.bfloat16 if bf16_out else torch.float32,
                          want_acc=not bf16_out and M * O * (C // g) < 4_000_000)
    compare_y(y, ref, C // g, out_eps=2.0 ** -8 if bf16_out else 0.0)


@pytest.mark.gpu
@pytest.mark.parametrize("M,C,O,g,bf16_out,with_bias", [s for s in _random_linear_shapes(60, seed=7) if s[1] <= 768][:16])
def test_fused_and_power_of_two_random_shapes(tdq, M, C, O, g, bf16_out, with_bias):
    rng = np.random.RandomState(M + 3 * C + 5 * O)
    x = (rng.normal(size=(M, C)) * np.exp(rng.normal(0, 1.0, size=(M, 1)))).astype(np.float32)
    w = (rng.normal(size=(O, C)) * 0.05).astype(np.float32)
    bias = rng.normal(size=(O,)).astype(np.float32) * 0.1 if with_bias else None
    dt = torch.bfloat16 if bf16_out else torch.float32
    xt, wc_ws = to_cuda(x), tdq.quantize_weight(to_cuda(w))
    b = None if bias is None else to_cuda(bias)
    # fused == the two calls, bit for bit (group size 32 is the fused path's)
    codes, scale = tdq.quantize_act(xt)
    y2 = tdq.w4a4_linear(codes, scale, *wc_ws, b, out_dtype=dt)
    y1 = tdq.quant_linear_fused(xt, *wc_ws, b, out_dtype=dt)
    assert torch.equal(y1.view(torch.int16 if bf16_out else torch.int32), y2.view(torch.int16 if bf16_out else torch.int32))
    # power-of-two steps at the drawn group size against the exact layer's oracle
    y, ref, _ = _pow2_case(tdq, x, False, w, g=g, bias=bias, out_dtype=dt)
    compare_y(y, ref, C, out_eps=2.0 ** -8 if bf16_out else 0.0)


# ------------------------------------------------------------------------------------------
# the launch configuration the benchmark times: steps replayed from a CUDA graph over rotating buffers

def test_full_size_step_replayed_from_a_graph_matches_oracle_on_sampled_rows(tdq):
    case = si.config(4)
    x = case.x.reshape(-1, case.C)
    M, C, O = x.shape[0], case.C, case.w.shape[0]
    nsets = 2
    xt = to_cuda(x, bf16=case.x_is_bf16)
    wc, ws = tdq.quantize_weight(to_cuda(case.w))
    codes = [torch.zeros((M, C // 2), dtype=torch.uint8, device="cuda") for _ in range(nsets)]
    scales = [torch.zeros((M, C // 32), dtype=torch.float32, device="cuda") for _ in range(nsets)]
    ys = [torch.zeros((M, O), dtype=torch.float32, device="cuda") for _ in range(nsets)]
    wsp = tdq.linear_workspace(M, C, O, 32, "cuda")
    params = tdq.default_act_params()

    def step(i):
        s = i % nsets
        tdq.quantize_act(xt, params, codes=codes[s], scale=scales[s])
        tdq.w4a4_linear(codes[s], scales[s], wc, ws, y=ys[s], workspace=wsp)

    step(0)
    torch.cuda.synchronize()
    y_eager = ys[0].clone()
    for t in codes + scales + ys:
        t.zero_()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i in range(2 * nsets):
            step(i)
    for t in codes + scales + ys:
        t.zero_()
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    st, detail = tdq.workspace_status(wsp)
    assert st == tdq.OK, "device wait ran out: 0x%x" % detail
    for s in range(nsets):
        assert torch.equal(ys[s].view(torch.int32), y_eager.view(torch.int32))      # every set, same bits as the eager call
    rng = np.random.default_rng(44)
    rows = np.unique(np.concatenate([rng.choice(M, 96, replace=False), [0, 127, 128, M - 1]]))
    xa = oracle.quantize_act(x[rows])
    wq = oracle.quantize_weight(case.w)
    ref = oracle.w4a4_linear(xa["codes"], xa["scale"], wq["codes"], wq["scale"])
    np.testing.assert_array_equal(codes[1].cpu().numpy()[rows], xa["codes"])
    np.testing.assert_array_equal(scales[1].cpu().numpy()[rows], xa["scale"])
    compare_y(ys[1].cpu().numpy()[rows], ref, C // 32)
