"""GPU parity at the configured sizes: every row of the large single-layer workloads, every layer of the
32-layer sweep at its batch size, a constructed set of rounding-boundary inputs, channel-major input through
the linear layer, and row shards against the unsharded call.  Everything goes through the C ABI (ctypes
binding of libtdq.so) and is compared with the CPU oracle under the rules of parity_utils."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from parity_utils import compare_quantizer, compare_y, to_cuda, unpack_codes

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tdq():
    from paper_2604_16855_b200 import tdq
    return tdq


def _f32(x_np, bf16):
    return si.bf16_bits_to_f32(x_np) if bf16 else x_np


# ---------------------------------------------------------------------------------------
# the two large single-layer workloads: quantizer -> linear layer, every row against the oracle

@pytest.mark.parametrize("idx", [3, 4])
def test_large_workloads_every_row(tdq, idx):
    case = si.config(idx)
    x = case.x.reshape(-1, case.C)
    K = case.C // 32
    xt = to_cuda(x, bf16=case.x_is_bf16)
    wc, ws = tdq.quantize_weight(to_cuda(case.w))
    codes, scale = tdq.quantize_act(xt)
    wsp = tdq.linear_workspace(x.shape[0], case.C, case.O, 32, "cuda")
    y = tdq.w4a4_linear(codes, scale, wc, ws, workspace=wsp)
    st, detail = tdq.workspace_status(wsp)
    assert st == tdq.OK, "device wait ran out: 0x%x" % detail
    xa = oracle.quantize_act(x)
    wq = oracle.quantize_weight(case.w)
    np.testing.assert_array_equal(codes.cpu().numpy(), xa["codes"])
    np.testing.assert_array_equal(scale.cpu().numpy(), xa["scale"])
    np.testing.assert_array_equal(wc.cpu().numpy(), wq["codes"])
    ref = oracle.w4a4_linear(xa["codes"], xa["scale"], wq["codes"], wq["scale"])
    worst, strict = compare_y(y.cpu().numpy(), ref, K)
    print("cfg%d, all %d rows: worst err/tol %.3f, %.6f of outputs within 1e-5 relative" % (idx, x.shape[0], worst, strict))
    assert strict > 0.99


# ---------------------------------------------------------------------------------------
# the 32-layer sweep at batch 8: every layer, quantizer and linear layer, and the fused call where it applies

@pytest.mark.parametrize("layer", list(range(32)))
def test_sweep_every_layer_at_batch_8(tdq, layer):
    case = si.config5_layer(layer, batch=8)
    x = case.x.reshape(-1, case.C)
    M, K = x.shape[0], case.C // 32
    xt = to_cuda(x, bf16=True)
    wc, ws = tdq.quantize_weight(to_cuda(case.w))
    codes, scale = tdq.quantize_act(xt)
    wsp = tdq.linear_workspace(M, case.C, case.O, 32, "cuda")
    y = tdq.w4a4_linear(codes, scale, wc, ws, workspace=wsp)
    st, detail = tdq.workspace_status(wsp)
    assert st == tdq.OK, "device wait ran out: 0x%x" % detail
    xa = oracle.quantize_act(x)
    wq = oracle.quantize_weight(case.w)
    rep = compare_quantizer(_f32(x, True), 32, xa, codes.cpu().numpy(), scale.cpu().numpy())
    assert rep["code_mismatch"] == 0 and rep["scale_exact_frac"] == 1.0, rep
    ref = oracle.w4a4_linear(xa["codes"], xa["scale"], wq["codes"], wq["scale"])
    worst, strict = compare_y(y.cpu().numpy(), ref, K)
    assert strict > 0.99
    if case.C <= 768:                            # the fused call keeps a row block's operand in shared memory
        yf = tdq.quant_linear_fused(xt, wc, ws)
        compare_y(yf.cpu().numpy(), ref, K)
    else:
        with pytest.raises(tdq.TdqError) as e:
            tdq.quant_linear_fused(xt, wc, ws)
        assert e.value.code == tdq.ERR_UNSUPPORTED
    print("layer %d (%d x %d -> %d): worst err/tol %.3f" % (layer, M, case.C, case.O, worst))


# ---------------------------------------------------------------------------------------
# rounding boundaries: inputs placed on and next to the half-integers of x / Delta

def _boundary_rows_fp32(n_rows, seed):
    """Rows of three groups whose step is set by the group's largest element c (a random binary32 mantissa and
    exponent): the other elements sit at (k + 1/2) * fl(c / 7), k = -7 .. 6, moved by 0, +-1 and +-2 ulp."""
    rng = np.random.default_rng(seed)
    c = (rng.uniform(1.0, 2.0, n_rows) * 2.0 ** rng.integers(-20, 20, n_rows)).astype(np.float32)
    delta = (c / np.float32(7.0)).astype(np.float32)
    vals = []
    for k in range(-7, 7):
        base = (np.float32(k + 0.5) * delta).astype(np.float32)
        for n in (-2, -1, 0, 1, 2):
            v = base.copy()
            for _ in range(abs(n)):
                v = np.nextafter(v, np.float32(np.inf if n > 0 else -np.inf), dtype=np.float32)
            vals.append(v)
    vals = np.stack(vals, 1)                       # [n_rows, 70]
    x = np.zeros((n_rows, 96), np.float32)
    for g in range(3):
        x[:, 32 * g] = c * (1 if g != 1 else -1)   # the group's largest magnitude
        take = vals[:, 24 * g: 24 * g + 24] if g < 2 else vals[:, 46:70]
        x[:, 32 * g + 1: 32 * g + 1 + take.shape[1]] = take
        x[:, 32 * g + 25: 32 * g + 32] = (rng.uniform(-1, 1, (n_rows, 7)).astype(np.float32) * c[:, None])
    return x


def _boundary_rows_zero_bin(n_rows, seed, bf16):
    """Groups in which the zero-bin bound is the active one: six small elements, the threshold element thr, odd
    multiples of thr (the half-integers of x / Delta, since Delta = 2 thr when 14 thr is exact) and their
    neighbours, and a few large elements that keep the other two bounds away."""
    rng = np.random.default_rng(seed)
    mant = rng.integers(8, 16, n_rows).astype(np.float32) if bf16 else rng.uniform(1.0, 2.0, n_rows).astype(np.float32)
    thr = (mant * np.float32(2.0) ** rng.integers(-12, 8, n_rows).astype(np.float32)).astype(np.float32)
    x = np.zeros((n_rows, 32), np.float32)
    x[:, :6] = thr[:, None] * rng.uniform(0.05, 0.9, (n_rows, 6)).astype(np.float32)
    x[:, 6] = thr
    odd = np.array([3, -3, 5, -5, 7, -7, 9, -9, 11, -11, 13, -13], np.float32)
    x[:, 7:19] = thr[:, None] * odd[None, :]
    nb = x[:, 7:13].copy()
    step = np.float32(2.0 ** -7) if bf16 else np.float32(2.0 ** -23)
    x[:, 19:25] = nb * (np.float32(1.0) + step)    # one unit in the last place above (bf16) or one ulp (fp32)
    x[:, 25:29] = x[:, 7:11] * (np.float32(1.0) - step)
    x[:, 29:32] = thr[:, None] * np.array([40.0, -60.0, 50.0], np.float32)[None, :]
    perm = rng.permuted(np.tile(np.arange(32), (n_rows, 1)), axis=1)
    return np.take_along_axis(x, perm, axis=1)


@pytest.mark.parametrize("kind", ["fp32_base", "fp32_zero_bin", "bf16_zero_bin"])
def test_quotients_on_rounding_boundaries(tdq, kind):
    bf16 = kind.startswith("bf16")
    if kind == "fp32_base":
        x = _boundary_rows_fp32(6000, 5)
        settings = [dict(flags=0), dict(flags=3)]
    else:
        x = _boundary_rows_zero_bin(20000, 9 if bf16 else 8, bf16)
        settings = [dict(flags=3), dict(flags=2)]
    xin = si.f32_to_bf16_bits(x) if bf16 else x
    xf = _f32(xin, bf16)
    for kw in settings:
        ref = oracle.quantize_act(xin, **kw)
        codes, scale = tdq.quantize_act(to_cuda(xin, bf16=bf16), tdq.act_params(**kw))
        torch.cuda.synchronize()
        rep = compare_quantizer(xf, 32, ref, codes.cpu().numpy(), scale.cpu().numpy())
        # how adversarial the set is: elements whose quotient lies within 4 ulp of a half-integer
        d = np.repeat(ref["scale"].astype(np.float64), 32, axis=1)
        cl = np.repeat(ref["clip"].astype(np.float64), 32, axis=1)
        r = np.clip(xf.astype(np.float64), -cl, cl) / d
        near = np.abs(np.abs(r - np.floor(r)) - 0.5) <= 4 * 2.0 ** -23 * np.maximum(np.abs(r), 1.0)
        print("%s %s: %d elements, %.1f %% within 4 ulp of a rounding boundary, %d code mismatches, scales exact %.6f"
              % (kind, kw, near.size, 100.0 * near.mean(), rep["code_mismatch"], rep["scale_exact_frac"]))
        assert near.mean() > 0.05
        assert rep["code_mismatch"] == 0 and rep["scale_exact_frac"] == 1.0


# ---------------------------------------------------------------------------------------
# channel-major input through the linear layer (a 1 x 1 convolution), against the oracle

@pytest.mark.parametrize("B,C,H,W,O,bf16", [(2, 64, 9, 16, 96, True), (1, 320, 24, 24, 320, True), (2, 128, 8, 8, 40, False)])
def test_channel_major_quantizer_feeds_the_linear_layer(tdq, B, C, H, W, O, bf16):
    rng = np.random.default_rng(B * 100 + C + O)
    sig = np.exp(rng.normal(0.0, 0.7, size=(B, 1, H, W)))
    x = (rng.normal(size=(B, C, H, W)) * sig).astype(np.float32)
    x[rng.random((B, C, H, W)) < 0.02] *= 30.0
    xin = si.f32_to_bf16_bits(x) if bf16 else x
    w = si.weights(rng, O, C)
    bias = rng.standard_normal(O).astype(np.float32) * 0.1
    codes, scale = tdq.quantize_act_nchw(to_cuda(xin, bf16=bf16))
    wc, ws = tdq.quantize_weight(to_cuda(w))
    y = tdq.w4a4_linear(codes, scale, wc, ws, to_cuda(bias))          # [B*H*W, O], token (b, h, w) in row (b*H + h)*W + w
    xa = oracle.quantize_act_nchw(xin)
    wq = oracle.quantize_weight(w)
    np.testing.assert_array_equal(codes.cpu().numpy(), xa["codes"])
    np.testing.assert_array_equal(scale.cpu().numpy(), xa["scale"])
    ref = oracle.w4a4_linear(xa["codes"], xa["scale"], wq["codes"], wq["scale"], bias=bias)
    compare_y(y.cpu().numpy(), ref, C // 32 + 1)
    # the rows are in token order: one position checked by plain indexing against the dequantized operands
    b, h, wq_pos = B - 1, H // 2, W - 1
    t = (b * H + h) * W + wq_pos
    xq = unpack_codes(xa["codes"])[t].astype(np.float64) * np.repeat(xa["scale"][t].astype(np.float64), 32)
    wd = unpack_codes(wq["codes"]).astype(np.float64) * wq["scale"].astype(np.float64)[:, None]
    np.testing.assert_allclose(y.cpu().numpy()[t], wd @ xq + bias, rtol=1e-4, atol=1e-5 * np.abs(wd @ xq).max())
    # and the dequantized token is the token at (b, :, h, w) of the map, within half a step per channel
    xf = _f32(xin, bf16)
    assert (np.abs(xq[:C] - np.clip(xf[b, :, h, wq_pos], -np.repeat(xa["clip"][t], 32)[:C], np.repeat(xa["clip"][t], 32)[:C]))
            <= 0.5000001 * np.repeat(xa["scale"][t], 32)[:C]).all()


# ---------------------------------------------------------------------------------------
# row shards: two ranges of rows through the path separately equal the unsharded call bit for bit

@pytest.mark.parametrize("idx,rows,split", [(2, 5000, 2176), (3, 3000, 1409), (1, 256, 100)])
def test_row_shards_equal_the_unsharded_call(tdq, idx, rows, split):
    case = si.config(idx)
    x = case.x.reshape(-1, case.C)[:rows]
    xt = to_cuda(x, bf16=case.x_is_bf16)
    wc, ws = tdq.quantize_weight(to_cuda(case.w))
    bias = torch.linspace(-0.5, 0.5, case.O, device="cuda")

    def path(xpart):
        codes, scale = tdq.quantize_act(xpart)
        return codes, scale, tdq.w4a4_linear(codes, scale, wc, ws, bias)

    c_all, s_all, y_all = path(xt)
    c0, s0, y0 = path(xt[:split])
    c1, s1, y1 = path(xt[split:].contiguous())
    assert torch.equal(torch.cat([c0, c1]), c_all)
    assert torch.equal(torch.cat([s0, s1]).view(torch.int32), s_all.view(torch.int32))
    assert torch.equal(torch.cat([y0, y1]).view(torch.int32), y_all.view(torch.int32))
    if case.C <= 768:
        yf0 = tdq.quant_linear_fused(xt[:split], wc, ws, bias)
        yf1 = tdq.quant_linear_fused(xt[split:].contiguous(), wc, ws, bias)
        assert torch.equal(torch.cat([yf0, yf1]).view(torch.int32), y_all.view(torch.int32))


# ---------------------------------------------------------------------------------------
# percentile base radius at any rank, with any zero-bin rank, on the fast kernels (ranks taken at run time)

@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("p,zr,flags", [(0.5, 0.2, 3), (0.75, 0.2, 3), (0.25, 0.1, 3), (0.04, 0.2, 3), (0.85, 0.5, 3), (0.6, 1.0, 3),
                                        (0.95, 0.4, 3), (0.7, 0.2, 1), (0.3, 0.3, 2), (0.5, 0.2, 0), (0.999, 0.03, 3)])
def test_any_pair_of_ranks_on_the_fast_kernels(tdq, bf16, p, zr, flags):
    n0 = None
    for x, stride_pad in ((si.config3().x.reshape(-1, 320)[:2000], 0), (si.edge_rows(C=64), 0), (si.dc_offset_tokens(M=700, C=96), 32)):
        if x.dtype == np.uint16:
            x = si.bf16_bits_to_f32(x)
        xin = si.f32_to_bf16_bits(x) if bf16 else x
        ref = oracle.quantize_act(xin, p=p, zr=zr, flags=flags)
        xt = to_cuda(xin, bf16=bf16)
        if stride_pad:                                # rows with a pitch: the strided fast kernel
            wide = torch.zeros((xt.shape[0], xt.shape[1] + stride_pad), dtype=xt.dtype, device="cuda")
            wide[:, : xt.shape[1]] = xt
            xt = wide[:, : x.shape[1]]
        codes, scale = tdq.quantize_act(xt, tdq.act_params(p=p, zr=zr, flags=flags))
        torch.cuda.synchronize()
        rep = compare_quantizer(_f32(xin, bf16), 32, ref, codes.cpu().numpy(), scale.cpu().numpy())
        assert rep["code_mismatch"] == 0 and rep["scale_exact_frac"] == 1.0, rep


# ---------------------------------------------------------------------------------------
# the affine output correction, folded into the layer's constants

@pytest.mark.parametrize("with_bias,with_shift,fused", [(True, True, False), (False, True, False), (True, False, True), (False, False, False)])
def test_affine_output_correction_folded_into_the_constants(tdq, with_bias, with_shift, fused):
    case = si.config3()
    x = case.x.reshape(-1, case.C)[:1300]
    rng = np.random.default_rng(17)
    O = case.O
    bias = rng.standard_normal(O).astype(np.float32) * 0.05 if with_bias else None
    a = (rng.uniform(0.5, 1.5, O) * rng.choice([-1.0, 1.0], O)).astype(np.float32)
    b = rng.standard_normal(O).astype(np.float32) * 0.1 if with_shift else None
    xt = to_cuda(x, bf16=True)
    wc, ws = tdq.quantize_weight(to_cuda(case.w))
    ws2, b2 = tdq.fold_output_affine(ws, None if bias is None else to_cuda(bias), to_cuda(a), None if b is None else to_cuda(b))
    if fused:
        y = tdq.quant_linear_fused(xt, wc, ws2, b2)
    else:
        codes, scale = tdq.quantize_act(xt)
        y = tdq.w4a4_linear(codes, scale, wc, ws2, b2)
    xa, wq = oracle.quantize_act(x), oracle.quantize_weight(case.w)
    ref = oracle.output_affine(oracle.w4a4_linear(xa["codes"], xa["scale"], wq["codes"], wq["scale"], bias=bias), a, b,
                               bias=np.zeros(O, np.float32) if bias is None else bias)
    # three more roundings than the plain layer (a_o s_o, a_o bias_o, + b_o), counted against the size of the terms
    compare_y(y.cpu().numpy(), ref, case.C // 32 + 3)


# ---------------------------------------------------------------------------------------
# fp16 output (rounded to nearest even from the float32 result), on both linear kernels and the fused call

@pytest.mark.parametrize("idx,rows,g,fused", [(3, 1500, 32, False), (3, 700, 64, False), (2, 3000, 32, True), (1, 256, 32, False)])
def test_fp16_output(tdq, idx, rows, g, fused):
    case = si.config(idx)
    x = case.x.reshape(-1, case.C)[:rows]
    bias = np.linspace(-0.3, 0.3, case.O).astype(np.float32)
    xt = to_cuda(x, bf16=case.x_is_bf16)
    wc, ws = tdq.quantize_weight(to_cuda(case.w), pad_to=g)
    p = tdq.act_params(g=g)
    if fused:
        y = tdq.quant_linear_fused(xt, wc, ws, to_cuda(bias), p, out_dtype=torch.float16)
    else:
        codes, scale = tdq.quantize_act(xt, p)
        y = tdq.w4a4_linear(codes, scale, wc, ws, to_cuda(bias), g=g, out_dtype=torch.float16)
        y32 = tdq.w4a4_linear(codes, scale, wc, ws, to_cuda(bias), g=g)
        assert torch.equal(y, y32.to(torch.float16))          # exactly the float32 result rounded once
    assert y.dtype == torch.float16
    xa, wq = oracle.quantize_act(x, g=g), oracle.quantize_weight(case.w, pad_to=g)
    ref = oracle.w4a4_linear(xa["codes"], xa["scale"], wq["codes"], wq["scale"], bias=bias, g=g)
    # one fp16 rounding on top of the float32 rule: 2^-11 relative, or half the spacing of fp16 subnormals (2^-24)
    # for the outputs of the low-amplitude tokens, which fall below fp16's smallest normal number
    yn = y.float().cpu().numpy().astype(np.float64)
    small = np.abs(ref["y_d"]) < 2.0 ** -14
    ref_n = dict(y_d=np.where(small, yn, ref["y_d"]), t_abs=ref["t_abs"])
    compare_y(yn, ref_n, case.C // g + 1, out_eps=2.0 ** -11)
    tol_small = np.maximum(1e-5 * np.abs(ref["y_d"]), (case.C // g + 3) * 2.0 ** -24 * ref["t_abs"]) + 2.0 ** -25
    assert (np.abs(yn - ref["y_d"])[small] <= tol_small[small]).all()


# ---------------------------------------------------------------------------------------
# one group per token with a contraction of two or more ring stages: the two MMA-issuing warps take the
# stages in turn, each into a TMEM accumulator of its own, and the promotion warps add the two integer sums.
# Even and odd numbers of stages, several tiles per CTA (both pairs of accumulators), ragged edges, resident and
# streamed operands.

@pytest.mark.parametrize("M,C,O,bf16_out", [(300, 256, 200, False), (20000, 384, 384, False), (700, 640, 130, True),
                                            (2100, 768, 1280, False), (129, 1024, 700, True), (5000, 128, 96, False),
                                            # operands streamed (K too long to stay resident): strips with 32-byte rows, written in passes
                                            (300, 2048, 200, False), (260, 4096, 130, True), (700, 2176, 100, False), (40000, 2048, 128, True),
                                            # K at which the operands stream with the usual strips but would stay resident with the small ones
                                            (300, 1152, 200, False), (2500, 1152, 64, True)])
def test_one_group_per_token_split_over_two_accumulators(tdq, M, C, O, bf16_out):
    rng = np.random.RandomState(M + 3 * C + O)
    x = (rng.normal(size=(M, C)) * np.exp(rng.normal(0, 1.0, size=(M, 1)))).astype(np.float32)
    w = (rng.normal(size=(O, C)) * 0.05).astype(np.float32)
    bias = rng.normal(size=(O,)).astype(np.float32) * 0.1
    xa, wq = oracle.quantize_act(x, g=C), oracle.quantize_weight(w, pad_to=C)
    xc, xs = to_cuda(xa["codes"]), to_cuda(xa["scale"])
    wc, ws = to_cuda(wq["codes"]), to_cuda(wq["scale"])
    want_acc = not bf16_out and M * O < 4_000_000
    acc = torch.full((M, O, 1), 12345, dtype=torch.int32, device="cuda") if want_acc else None
    wsp = tdq.linear_workspace(M, C, O, C, "cuda")
    y = tdq.w4a4_linear(xc, xs, wc, ws, to_cuda(bias), g=C, out_dtype=torch.bfloat16 if bf16_out else torch.float32,
                        acc_debug=acc, workspace=wsp)
    st, detail = tdq.workspace_status(wsp)
    assert st == tdq.OK, "device wait ran out: 0x%x" % detail
    ref = oracle.w4a4_linear(xa["codes"], xa["scale"], wq["codes"], wq["scale"], bias=bias, g=C, want_acc=want_acc)
    if want_acc:
        np.testing.assert_array_equal(acc.cpu().numpy(), ref["acc"])      # the sum of the two accumulators, bit-exact
    compare_y(y.float().cpu().numpy(), ref, 2, out_eps=2.0 ** -8 if bf16_out else 0.0)
    # a second call on the same workspace reproduces the first bit for bit (the accumulator pairs alternate per tile)
    y2 = tdq.w4a4_linear(xc, xs, wc, ws, to_cuda(bias), g=C, out_dtype=y.dtype, workspace=wsp)
    assert torch.equal(y, y2)


# ---------------------------------------------------------------------------------------
# Exactness of the accumulators on constructed codes: the largest sums a group can produce and sums with busy
# low bits (a constant operand against varied codes), on both operand routes (E4M3 with an fp32 accumulator up
# to 128 codes per group, int8 with an int32 accumulator beyond), resident and streamed operands.

def _pack_codes(q):
    u = (q.astype(np.int16) & 15).astype(np.uint8)
    return (u[:, 0::2] | (u[:, 1::2] << 4)).astype(np.uint8)


@pytest.mark.parametrize("M,C,O,g", [(200, 256, 130, 32), (200, 512, 130, 64), (130, 1024, 100, 128), (130, 4096, 128, 128),
                                     (128, 1024, 128, 256), (150, 768, 96, 768), (140, 4096, 128, 4096)])
def test_group_sums_are_exact_on_extreme_codes(tdq, M, C, O, g):
    rng = np.random.RandomState(g + C)
    for kind in ("all -8", "all 7", "7 against varied", "alternating 7 / -8", "random"):
        if kind == "all -8":
            qx, qw = np.full((M, C), -8, np.int8), np.full((O, C), -8, np.int8)
        elif kind == "all 7":
            qx, qw = np.full((M, C), 7, np.int8), np.full((O, C), 7, np.int8)
        elif kind == "7 against varied":
            qx, qw = np.full((M, C), 7, np.int8), rng.randint(1, 8, size=(O, C)).astype(np.int8)
        elif kind == "alternating 7 / -8":
            qx = np.where(np.arange(C)[None, :] % 2 == 0, 7, -8).astype(np.int8).repeat(M, 0)
            qw = rng.randint(-8, 8, size=(O, C)).astype(np.int8)
        else:
            qx, qw = rng.randint(-8, 8, size=(M, C)).astype(np.int8), rng.randint(-8, 8, size=(O, C)).astype(np.int8)
        xs = np.ones((M, C // g), np.float32)
        ws = np.ones((O,), np.float32)
        acc = torch.full((M, O, C // g), 12345, dtype=torch.int32, device="cuda")
        wsp = tdq.linear_workspace(M, C, O, g, "cuda")
        y = tdq.w4a4_linear(to_cuda(_pack_codes(qx)), to_cuda(xs), to_cuda(_pack_codes(qw)), to_cuda(ws), g=g, acc_debug=acc, workspace=wsp)
        st, detail = tdq.workspace_status(wsp)
        assert st == tdq.OK, "device wait ran out: 0x%x" % detail
        ref = np.einsum("mkg,okg->mok", qx.reshape(M, C // g, g).astype(np.int64), qw.reshape(O, C // g, g).astype(np.int64))
        np.testing.assert_array_equal(acc.cpu().numpy().astype(np.int64), ref, err_msg=kind)
        # unit steps and unit channel scales: y is the integer sum over the groups, exact in binary32 below 2^24
        np.testing.assert_array_equal(y.cpu().numpy().astype(np.int64), ref.sum(axis=2), err_msg=kind)


# ------------------------------------------------------------------------------------------
# the power-of-two variant's operand bytes: every code value at every shift against the row's largest
# step, the truncated ones included.  One-hot weight rows leave a single product per output, so every
# expected value is exact in binary32 and the comparison is bit for bit.

@pytest.mark.parametrize("C,g", [(128, 32), (256, 64), (256, 128), (768, 768)])
def test_power_of_two_operand_is_exact_for_every_code_and_shift(tdq, C, g):
    rng = np.random.RandomState(C + g)
    M, O, Kg = 300, C, C // g
    qx = ((np.arange(C)[None, :] + np.arange(M)[:, None] * 5) % 16 - 8).astype(np.int8)
    drop = rng.randint(0, 22, size=(M, Kg))                # binades below the row's largest step
    drop[np.arange(M), rng.randint(0, Kg, size=M)] = 0
    drop[:23, 0] = 0
    if Kg > 1:
        drop[:23, 1] = np.arange(23)                       # every shift from 14 down to -8 occurs
    top = rng.randint(-12, 6, size=(M, 1))
    xs = np.exp2(top - drop).astype(np.float32)
    qw = np.zeros((O, C), np.int8)
    nz = np.array([7, -8, 1, -1, 3, -5, 6, -2, 4, -7], np.int8)
    qw[np.arange(O), np.arange(C)] = nz[np.arange(O) % len(nz)]
    ws = np.exp2(-(np.arange(O) % 5)).astype(np.float32)
    wsp = tdq.linear_workspace(M, C, O, g, "cuda")
    y = tdq.w4a4_linear_pow2(to_cuda(_pack_codes(qx)), to_cuda(xs), to_cuda(_pack_codes(qw)), to_cuda(ws), None,
                             g=g, out_dtype=torch.float32, workspace=wsp)
    st, detail = tdq.workspace_status(wsp)
    assert st == tdq.OK, "status 0x%x" % detail
    # s = 14 - drop; a code keeps |q| >> max(-s, 0) (towards zero) and its step
    shr = np.maximum(drop - 14, 0).repeat(g, axis=1)
    kept = np.sign(qx.astype(np.int64)) * (np.abs(qx.astype(np.int64)) >> shr)
    v = kept.astype(np.float64) * np.exp2(shr) * xs.astype(np.float64).repeat(g, axis=1)
    want = v * (np.diag(qw).astype(np.float64) * ws.astype(np.float64))[None, :]
    np.testing.assert_array_equal(y.cpu().numpy().astype(np.float64), want)
