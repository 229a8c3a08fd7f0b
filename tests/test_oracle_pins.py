"""Pins for the CPU oracle: what the paper and plain mathematics fix, checked on the host.

Nothing here touches the CUDA library.  Each test is written so that a plausible slip in
the oracle (a dropped bound, the sample instead of the population deviation, an off-by-one
rank, half-away-from-zero rounding, swapped nibbles, a transposed weight) makes it fail.
"""
import os

import numpy as np
import pytest

import oracle
import synth_inputs as si

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
F32_EPS = 2.0 ** -23


def _groups(x, g):
    """float64 view [M, K, g] of x [M, C] zero-padded on the channel axis (Eq. 5)."""
    M, C = x.shape
    K = -(-C // g)
    xp = np.zeros((M, K * g), np.float64)
    xp[:, :C] = x
    return xp.reshape(M, K, g)


def _cases_default():
    c1 = si.config1()
    x1 = c1.x.reshape(-1, c1.C)
    c2 = si.config2()
    x2 = c2.x_f32().reshape(-1, c2.C)[:2048]
    return [("cfg1", x1, c1.x.reshape(-1, c1.C)), ("cfg2", x2, c2.x.reshape(-1, c2.C)[:2048])]


# ---------------------------------------------------------------------------------------
# rank convention (Supp. S2.2)

def test_rank_examples_golden():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "rank_examples.txt")) if l.strip() and l[0] != "#"]
    assert rows[0][:3] == ["32", "0.99", "32"]
    for g, frac, k, _src in rows:
        assert oracle.rank(float(frac), int(g)) == int(k), (g, frac, k)


def test_percentile_099_is_group_max():
    x = si.config1().x.reshape(-1, 64)
    a = oracle.quantize_act(x, g=32, p=0.99, flags=0)
    b = oracle.quantize_act(x, g=32, p=1.0, flags=0)
    np.testing.assert_array_equal(a["clip"], b["clip"])
    np.testing.assert_array_equal(a["clip"], np.maximum(np.abs(_groups(x, 32)).max(-1), 1e-8).astype(np.float32))


def test_percentile_base_radius_is_order_statistic():
    x = si.config1().x.reshape(-1, 64)
    out = oracle.quantize_act(x, g=32, p=0.9, flags=0)       # k = ceil(28.8) = 29
    srt = np.sort(np.abs(_groups(x, 32)), axis=-1)
    np.testing.assert_array_equal(out["clip"], srt[..., 28].astype(np.float32))


def test_zr_one_never_binds_c2():
    x = si.config1().x.reshape(-1, 64)
    out = oracle.quantize_act(x, zr=1.0)
    assert not (out["active"] == 2).any()


# ---------------------------------------------------------------------------------------
# rounding convention

def test_round_half_to_even_golden_group():
    lines = [l for l in open(os.path.join(GOLDEN, "round_half_even_group.txt")) if l.strip() and l[0] != "#"]
    x = np.array([float(v) for v in lines[0].split()], np.float32)[None, :]
    want = np.array([int(v) for v in lines[1].split()], np.int8)[None, :]
    out = oracle.quantize_act(x, g=8, flags=0)
    assert out["scale"][0, 0] == np.float32(1.0)
    np.testing.assert_array_equal(out["q"], want)


def test_packing_low_nibble_is_even_channel():
    x = np.array([[7, -7, 1, -1, 0, 3, -3, 2]], np.float32)
    out = oracle.quantize_act(x, g=8, flags=0)
    np.testing.assert_array_equal(out["q"][0], [7, -7, 1, -1, 0, 3, -3, 2])
    want = [(7 & 15) | ((-7 & 15) << 4), (1 & 15) | ((-1 & 15) << 4), 0 | (3 << 4), (-3 & 15) | (2 << 4)]
    np.testing.assert_array_equal(out["codes"][0], np.array(want, np.uint8))


# ---------------------------------------------------------------------------------------
# Lemma 1, Proposition 1, zero-bin statement, code range

@pytest.mark.parametrize("tau,zr", [(1.0, 0.2), (0.5, 0.2), (0.25, 0.1), (1.0, 0.5)])
def test_lemma1_bounds_hold_on_every_group(tau, zr):
    xs = [c[1] for c in _cases_default()] + [si.dc_offset_tokens(), si.edge_rows()[4:9]]
    for x in xs:
        g = 32
        out = oracle.quantize_act(x, g=g, tau=tau, zr=zr)
        G = _groups(x, g)
        sigma = G.std(axis=-1) + 1e-12                      # population deviation, float64
        k = oracle.rank(zr, g)
        thr = np.sort(np.abs(G), axis=-1)[..., k - 1]
        delta = out["scale"].astype(np.float64)
        floored = out["clip"] <= np.float32(7e-8)           # step or radius floor reached
        ok1 = delta <= tau * sigma * (1 + 8 * F32_EPS)
        ok2 = delta / 2 <= thr * (1 + 8 * F32_EPS)
        assert (ok1 | floored).all()
        assert (ok2 | floored).all()
        # the projected radius never exceeds the base radius (Eq. 12)
        assert (out["clip"].astype(np.float64) <= np.maximum(np.abs(G).max(-1), 1e-8) * (1 + F32_EPS)).all()
        # zero-bin mass bound up to the rank slack: #{|x| <= Delta/2} <= #{|x| <= thr}
        zero_mass = (np.abs(G) <= delta[..., None] / 2).sum(-1)
        rank_mass = (np.abs(G) <= thr[..., None]).sum(-1)
        assert ((zero_mass <= rank_mass) | floored).all()


def test_c1_binds_on_dc_offset_and_never_on_zero_mean_at_tau1():
    out = oracle.quantize_act(si.dc_offset_tokens())
    assert (out["active"] == 1).mean() > 0.2
    x = si.config1().x.reshape(-1, 64)
    out = oracle.quantize_act(x)
    # Samuelson: max|x - mean| <= sqrt(g-1) sigma < 7 sigma, so C1 is idle unless the mean is large
    assert (out["active"] == 1).mean() < 0.01
    assert 0.05 < (out["active"] == 2).mean() < 0.5


def test_prop1_rounding_error_and_zero_bin_and_range():
    for _name, x, _raw in _cases_default():
        out = oracle.quantize_act(x)
        G = _groups(x, 32)
        q = out["q"].reshape(G.shape).astype(np.float64)
        delta = out["scale"].astype(np.float64)[..., None]
        c = out["clip"].astype(np.float64)[..., None]
        xt = np.clip(G, -c, c)
        err = np.abs(xt - q * delta)
        assert (err <= delta / 2 * (1 + 1e-6)).all()                       # Prop. 1, sup norm
        assert (np.sqrt((err ** 2).sum(-1)) <= np.sqrt(32) * delta[..., 0] / 2 * (1 + 1e-6)).all()
        assert q.min() >= -8 and q.max() <= 7
        a = np.abs(G)
        assert (q[a < delta / 2 * (1 - 1e-6)] == 0).all()                  # x_hat = 0 iff |x| <= Delta/2
        assert (q[a > delta / 2 * (1 + 1e-6)] != 0).all()
        assert (np.sign(q) * np.sign(G) >= 0).all()


def test_codes_unpack_to_q():
    x = si.config1().x.reshape(-1, 64)
    out = oracle.quantize_act(x)
    lo = (out["codes"] & 0xF).astype(np.int16)
    hi = (out["codes"] >> 4).astype(np.int16)
    lo = np.where(lo >= 8, lo - 16, lo)
    hi = np.where(hi >= 8, hi - 16, hi)
    np.testing.assert_array_equal(np.stack([lo, hi], -1).reshape(out["q"].shape), out["q"])


# ---------------------------------------------------------------------------------------
# brute-force projection on tiny groups (Eq. 12 is the largest feasible radius)

def _feasible(c, a_sorted, sigma, c_base, tau, k):
    # c <= c_base, Delta/sigma <= tau, and Delta/2 <= k-th smallest magnitude (Eq. 10, 11)
    # (a 1e-12 slack keeps the exact candidates 7 tau sigma and 14 a_i feasible under float64 rounding)
    s = 1 - 1e-12
    return c * s <= c_base and c * s / 7.0 <= tau * sigma and c * s / 14.0 <= a_sorted[k - 1]


@pytest.mark.parametrize("g", [4, 8])
def test_bruteforce_clip_search_agrees_with_projection(g):
    rng = np.random.default_rng(5)
    x = rng.standard_t(3, size=(300, g)) * np.exp(rng.normal(0, 1, size=(300, 1)))
    x[::3] += rng.uniform(2, 5, size=(100, 1))               # some groups where C1 binds
    x = x.astype(np.float32)
    for tau, zr in [(1.0, 0.5), (0.5, 0.3), (0.3, 0.8)]:
        out = oracle.quantize_act(x, g=g, tau=tau, zr=zr)
        k = oracle.rank(zr, g)
        for m in range(x.shape[0]):
            xv = x[m].astype(np.float64)
            a = np.sort(np.abs(xv))
            sigma = xv.std() + 1e-12
            c_base = a[-1]
            grid = np.unique(np.concatenate([np.linspace(0, c_base, 4001)[1:], 14 * a, [7 * tau * sigma, c_base]]))
            feas = [c for c in grid if _feasible(c, a, sigma, c_base, tau, k)]
            best = max(feas) if feas else 0.0
            got = float(out["clip"][m, 0])
            assert got == pytest.approx(max(best, 1e-8), rel=2e-6), (m, tau, zr)
            which = int(np.argmin([c_base, 7 * tau * sigma, 14 * a[k - 1]]))
            vals = sorted([c_base, 7 * tau * sigma, 14 * a[k - 1]])
            if vals[1] > vals[0] * (1 + 1e-5):
                assert out["active"][m, 0] == which


# ---------------------------------------------------------------------------------------
# reductions to textbook quantizers

def test_single_group_is_per_tensor_absmax_quantizer():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((1, 96)).astype(np.float32) * 3
    out = oracle.quantize_act(x, g=96, flags=0)
    step = np.float32(np.abs(x).max()) / np.float32(7)
    want = np.clip(np.rint(x / step), -8, 7).astype(np.int8)
    assert out["scale"][0, 0] == step
    np.testing.assert_array_equal(out["q"], want)


def test_group_equal_to_row_is_per_token_quantizer_and_dstg_only_scales():
    x = si.config1().x.reshape(-1, 64)
    out = oracle.quantize_act(x, g=64, flags=0)
    step = (np.abs(x).max(-1) / np.float32(7)).astype(np.float32)
    np.testing.assert_array_equal(out["scale"][:, 0], np.maximum(step, np.float32(1e-8)))
    np.testing.assert_array_equal(out["q"], np.clip(np.rint(x / step[:, None]), -8, 7).astype(np.int8))
    out32 = oracle.quantize_act(x, g=32, flags=0)
    step32 = (np.abs(x.reshape(-1, 2, 32)).max(-1) / np.float32(7)).astype(np.float32)
    np.testing.assert_array_equal(out32["scale"], step32)


def test_constraint_switches():
    x = si.dc_offset_tokens(M=64)
    both = oracle.quantize_act(x)
    c1 = oracle.quantize_act(x, flags=oracle.ENABLE_C1)
    c2 = oracle.quantize_act(x, flags=oracle.ENABLE_C2)
    none = oracle.quantize_act(x, flags=0)
    np.testing.assert_array_equal(both["clip"], np.minimum(c1["clip"], c2["clip"]))
    assert (c1["clip"] <= none["clip"]).all() and (c2["clip"] <= none["clip"]).all()
    assert not (c1["active"] == 2).any() and not (c2["active"] == 1).any()


# ---------------------------------------------------------------------------------------
# padding and degenerate groups

def test_padding_participates_and_degenerate_groups():
    rng = np.random.default_rng(9)
    x = rng.standard_normal((5, 48)).astype(np.float32)
    out = oracle.quantize_act(x, g=32)
    assert out["q"].shape == (5, 64) and out["scale"].shape == (5, 2)
    # second group: 16 real + 16 zero channels, so the rank-7 magnitude is 0 and c, Delta hit 1e-8
    assert (out["scale"][:, 1] == np.float32(1e-8)).all()
    assert (out["clip"][:, 1] == np.float32(1e-8)).all()
    np.testing.assert_array_equal(out["q"][:, 48:], 0)
    np.testing.assert_array_equal(out["q"][:, 32:48], np.sign(x[:, 32:]).astype(np.int8))
    # first group is the same as quantizing the first 32 channels alone
    alone = oracle.quantize_act(np.ascontiguousarray(x[:, :32]), g=32)
    np.testing.assert_array_equal(out["q"][:, :32], alone["q"])
    # with the constraints off the padded group keeps its own max
    off = oracle.quantize_act(x, g=32, flags=0)
    np.testing.assert_array_equal(off["clip"][:, 1], np.abs(x[:, 32:]).max(-1))

    z = np.zeros((2, 32), np.float32)
    oz = oracle.quantize_act(z)
    assert (oz["scale"] == np.float32(1e-8)).all() and (oz["q"] == 0).all()
    cst = np.full((1, 32), 2.5, np.float32)
    oc = oracle.quantize_act(cst)            # sigma = 1e-12, so C1 drives c to the floor
    assert oc["active"][0, 0] == 1 and oc["scale"][0, 0] == np.float32(1e-8)
    assert (oc["q"] == 1).all()


def test_row_stride_and_bf16_input():
    c2 = si.config2()
    bits = c2.x.reshape(-1, 64)[:64]
    a = oracle.quantize_act(bits)
    b = oracle.quantize_act(si.bf16_bits_to_f32(bits))
    for key in a:
        np.testing.assert_array_equal(a[key], b[key])
    wide = np.full((64, 80), 0x7F7F, np.uint16)            # junk beyond the 64 real channels
    wide[:, :64] = bits
    c = oracle.quantize_act(wide, C=64)
    for key in a:
        np.testing.assert_array_equal(a[key], c[key])


def test_bf16_rounding_helper_is_nearest_even():
    v = np.array([1.0, 1.00390625, 1.005859375, 1.01171875, -2.5, 3.0e38, 1e-40], np.float32)
    bits = si.f32_to_bf16_bits(v)
    back = si.bf16_bits_to_f32(bits)
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7 -> even (1.0); 1 + 3*2^-9 rounds up to 1 + 2^-7;
    # 1 + 3*2^-8 is a tie between 1+2^-7 (odd) and 1+2^-6 (even) -> 1 + 2^-6
    np.testing.assert_array_equal(back[:5], np.array([1.0, 1.0, 1.0078125, 1.015625, -2.5], np.float32))


# ---------------------------------------------------------------------------------------
# weight quantizer (Eq. 4)

def test_weight_quantizer_absmax_per_output_channel():
    w = si.config1().w
    out = oracle.quantize_weight(w, pad_to=32)
    s = (np.abs(w).max(-1) / np.float32(7)).astype(np.float32)
    np.testing.assert_array_equal(out["scale"], s)
    np.testing.assert_array_equal(out["q"], np.clip(np.rint(w / s[:, None]), -8, 7).astype(np.int8))
    assert np.abs(out["q"]).max(-1).min() == 7               # every row reaches +-7 at its absmax
    assert (np.abs(w - out["q"] * s[:, None].astype(np.float64)) <= s[:, None] / 2 * (1 + 1e-6)).all()
    w2 = np.ascontiguousarray(w[:, :40])
    o2 = oracle.quantize_weight(w2, pad_to=32)
    assert o2["q"].shape == (64, 64) and (o2["q"][:, 40:] == 0).all()
    z = oracle.quantize_weight(np.zeros((2, 32), np.float32))
    assert (z["scale"] == np.float32(1e-8)).all() and (z["q"] == 0).all()


# ---------------------------------------------------------------------------------------
# linear layer (Alg. S1 step 10)

@pytest.mark.parametrize("C,O,g", [(64, 64, 32), (100, 24, 32), (64, 16, 64), (96, 40, 16)])
def test_linear_equals_float64_product_of_dequantized_operands(C, O, g):
    rng = np.random.default_rng(C + O)
    x = si.token_mixture(rng, 1, 50, C, sigma_log_std=0.5, bg_frac=0.1, bg_nu=3.0, bg_amp=20.0).reshape(-1, C)
    w = si.weights(rng, O, C)
    bias = rng.standard_normal(O).astype(np.float32)
    xa = oracle.quantize_act(x, g=g)
    wq = oracle.quantize_weight(w, pad_to=g)
    out = oracle.w4a4_linear(xa["codes"], xa["scale"], wq["codes"], wq["scale"], bias=bias, g=g, want_acc=True)
    K = xa["scale"].shape[1]
    x_hat = (xa["q"].reshape(-1, K, g) * xa["scale"].astype(np.float64)[..., None]).reshape(-1, K * g)
    w_hat = wq["q"] * wq["scale"].astype(np.float64)[:, None]
    want = x_hat @ w_hat.T + bias.astype(np.float64)           # y = Linear(x_hat, W_hat)
    scale_ref = np.abs(x_hat) @ np.abs(w_hat).T + np.abs(bias)
    assert (np.abs(out["y_d"] - want) <= 1e-12 * scale_ref + 1e-300).all()
    np.testing.assert_array_equal(out["y"], out["y_d"].astype(np.float32))
    acc = np.einsum("mkg,okg->mok", xa["q"].reshape(-1, K, g).astype(np.int64),
                    wq["q"].reshape(O, K, g).astype(np.int64))
    np.testing.assert_array_equal(out["acc"], acc.astype(np.int32))
    assert np.abs(out["acc"]).max() <= g * 7 * 8
    t_abs = (np.abs(acc) * xa["scale"].astype(np.float64)[:, None, :]).sum(-1) * wq["scale"].astype(np.float64)
    np.testing.assert_allclose(out["t_abs"], t_abs, rtol=1e-12)
    # a transposed or mis-indexed weight would break this asymmetric check
    nb = oracle.w4a4_linear(xa["codes"], xa["scale"], wq["codes"], wq["scale"], g=g)
    np.testing.assert_allclose(nb["y_d"], want - bias, rtol=0, atol=float(1e-12 * scale_ref.max()))


def test_output_affine_is_a_diagonal_layer_after_the_linear_layer():
    """The affine correction (Supp. S1.1): against a float64 product with a diagonal matrix appended; the identity
    and pure-shift special cases; a swapped multiplier and shift, or a per-row instead of per-column vector, fail."""
    rng = np.random.default_rng(5)
    C, O = 96, 40
    x = si.token_mixture(rng, 1, 30, C, sigma_log_std=0.5, bg_frac=0.1, bg_nu=3.0, bg_amp=20.0).reshape(-1, C)
    w = si.weights(rng, O, C)
    bias = rng.standard_normal(O).astype(np.float32)
    a = rng.uniform(0.5, 1.5, O).astype(np.float32) * rng.choice([-1.0, 1.0], O).astype(np.float32)
    b = rng.standard_normal(O).astype(np.float32)
    xa, wq = oracle.quantize_act(x), oracle.quantize_weight(w)
    ref = oracle.w4a4_linear(xa["codes"], xa["scale"], wq["codes"], wq["scale"], bias=bias)
    out = oracle.output_affine(ref, a, b)
    K = xa["scale"].shape[1]
    x_hat = (xa["q"].reshape(-1, K, 32) * xa["scale"].astype(np.float64)[..., None]).reshape(-1, K * 32)
    w_hat = wq["q"] * wq["scale"].astype(np.float64)[:, None]
    want = (x_hat @ w_hat.T + bias.astype(np.float64)) @ np.diag(a.astype(np.float64)) + b.astype(np.float64)
    size = (np.abs(x_hat) @ np.abs(w_hat).T + np.abs(bias)) * np.abs(a) + np.abs(b)
    assert (np.abs(out["y_d"] - want) <= 1e-12 * size).all()
    np.testing.assert_array_equal(out["y"], out["y_d"].astype(np.float32))
    np.testing.assert_allclose(out["t_abs"], np.abs(a.astype(np.float64)) * ref["t_abs"], rtol=1e-15)
    same = oracle.output_affine(ref, np.ones(O, np.float32))
    np.testing.assert_array_equal(same["y_d"], ref["y_d"])
    shift = oracle.output_affine(ref, np.ones(O, np.float32), b)
    np.testing.assert_array_equal(shift["y_d"], ref["y_d"] + b.astype(np.float64))
    assert np.abs(oracle.output_affine(ref, b, a)["y_d"] - want).max() > 1e-3


def test_channel_major_wrapper_is_the_per_token_definition():
    """quantize_act_nchw must treat x[b, :, h, w] as one token (Supp. S1.1's 4-D branch), with token
    index (b*H + h)*W + w: checked token by token with plain indexing, no transpose."""
    rng = np.random.RandomState(5)
    B, C, H, W = 2, 64, 3, 5
    x = rng.normal(size=(B, C, H, W)).astype(np.float32)
    out = oracle.quantize_act_nchw(x)
    for b in range(B):
        for h in range(H):
            for w in range(W):
                one = oracle.quantize_act(np.array([x[b, c, h, w] for c in range(C)], np.float32)[None, :])
                t = (b * H + h) * W + w
                np.testing.assert_array_equal(out["codes"][t], one["codes"][0])
                np.testing.assert_array_equal(out["scale"][t], one["scale"][0])


def test_fixed_radius_control_against_the_token_group_path_and_its_bounds():
    """Pins for quantize_act_fixed.  (a) When every group's largest magnitude equals the fixed radius, the
    token-group quantizer without DCRP (flags = 0) chooses exactly that radius itself, so both must give the
    same codes and steps.  (b) Inside the radius the reconstruction error is at most half a step, outside
    the codes saturate at +-7, zeros stay zero."""
    rng = np.random.RandomState(3)
    M, C, g, radius = 40, 96, 32, 2.5
    x = rng.uniform(-radius, radius, size=(M, C)).astype(np.float32)
    x[:, ::g] = np.where(rng.rand(M, C // g) < 0.5, radius, -radius).astype(np.float32)   # plant the maximum in each group
    fixed = oracle.quantize_act_fixed(x, radius, g=g)
    dstg = oracle.quantize_act(x, g=g, flags=0)
    np.testing.assert_array_equal(fixed["codes"], dstg["codes"])
    np.testing.assert_array_equal(fixed["scale"], dstg["scale"])
    delta = np.float32(radius) / np.float32(7.0)
    assert np.all(fixed["scale"] == delta)
    assert np.abs(fixed["q"].astype(np.float64) * float(delta) - x).max() <= float(delta) / 2 * (1 + 1e-6)
    y = np.array([[0.0, 10.0, -10.0, radius * 1.0001] + [0.0] * 28], np.float32)
    out = oracle.quantize_act_fixed(y, radius, g=g)
    assert list(out["q"][0, :4]) == [0, 7, -7, 7]
    with pytest.raises(ValueError):
        oracle.quantize_act_fixed(y, 0.0)


def test_power_of_two_step_variant_keeps_the_bounds_and_only_shrinks_the_range():
    """Pins for the POW2_STEP variant: every step is a power of two with Delta/2 < Delta' <= Delta of the
    paper's quantizer, c' = 7 Delta' <= c (so both DCRP bounds, which are upper bounds on c, still hold), and
    the codes are what that grid gives: rint(clip(x, +-c') / Delta'), a division that is exact."""
    case = si.config2()
    x = case.x_f32().reshape(-1, case.C)[:800]
    base = oracle.quantize_act(x)
    pow2 = oracle.quantize_act(x, flags=oracle.ENABLE_C1 | oracle.ENABLE_C2 | oracle.POW2_STEP)
    d, dp = base["scale"].astype(np.float64), pow2["scale"].astype(np.float64)
    mant, _ = np.frexp(dp)
    assert np.all(mant == 0.5)                                  # powers of two
    assert np.all(dp <= d) and np.all(dp > d / 2)
    assert np.all(pow2["clip"].astype(np.float64) == 7.0 * dp)
    assert np.all(pow2["clip"] <= base["clip"])
    K = case.C // 32
    xg = x.astype(np.float64).reshape(-1, K, 32)
    c = pow2["clip"].astype(np.float64)[:, :, None]
    want = np.clip(np.rint(np.clip(xg, -c, c) / dp[:, :, None]), -8, 7).reshape(x.shape[0], -1)
    np.testing.assert_array_equal(pow2["q"], want.astype(np.int8))
