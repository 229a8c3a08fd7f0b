"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module holds no quantizer arithmetic.  It only draws random numbers (numpy's
PCG64, fixed seeds) in the shapes and value distributions of the five benchmark
workloads: heavy-tailed token activations of Transformer encoders for camouflaged
object detection (most tokens Gaussian with a log-normal per-token scale, a
minority of background tokens Student-t with a large amplitude, optionally a few
thin, structured, low-amplitude "boundary" tokens) and N(0, 0.02) weights.  They
stand in for the real CFRN / ESCNet activations, which need the trained models and
the COD datasets.

bf16 tensors are returned as uint16 bit patterns (numpy has no bf16); the rounding
from float32 is round-to-nearest-even, done once here so that every consumer reads
the same bits.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

DEFAULT_G = 32
DEFAULT_TAU = 1.0
DEFAULT_ZR = 0.2


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(a, np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << 16).view(np.float32)


@dataclass
class LinearCase:
    """One quantize -> W4A4-linear problem."""
    name: str
    x: np.ndarray            # [B, N, C] float32, or uint16 holding bf16 bits
    w: np.ndarray            # [O, I] float32
    x_is_bf16: bool
    g: int = DEFAULT_G
    tau: float = DEFAULT_TAU
    zr: float = DEFAULT_ZR
    bias: np.ndarray | None = None
    meta: dict = field(default_factory=dict)

    @property
    def M(self) -> int:
        return int(np.prod(self.x.shape[:-1]))

    @property
    def C(self) -> int:
        return int(self.x.shape[-1])

    @property
    def O(self) -> int:
        return int(self.w.shape[0])

    def x_f32(self) -> np.ndarray:
        return bf16_bits_to_f32(self.x) if self.x_is_bf16 else self.x


def token_mixture(rng, B, N, C, *, sigma_log_std, bg_frac, bg_nu, bg_amp,
                  outlier_frac=0.0, outlier_gain=1.0, boundary_frac=0.0):
    """Heavy-tailed token activations [B, N, C] in float32.

    Per token: with probability bg_frac a background token bg_amp * t_nu (iid Student-t);
    otherwise N(0, sigma_t^2) with ln sigma_t ~ N(0, sigma_log_std^2).  outlier_frac of
    the tokens are multiplied by outlier_gain.  boundary_frac of the tokens are replaced
    by a thin structured row 0.05 * (cos(2 pi f c / C + phi) + 0.1 N(0,1)), f in {1,2,3}.
    """
    T = B * N
    sigma_t = np.exp(rng.normal(0.0, sigma_log_std, size=T))
    x = rng.standard_normal(size=(T, C)) * sigma_t[:, None]
    if bg_frac > 0:
        is_bg = rng.random(T) < bg_frac
        nbg = int(is_bg.sum())
        if nbg:
            x[is_bg] = bg_amp * rng.standard_t(bg_nu, size=(nbg, C))
    if outlier_frac > 0:
        is_out = rng.random(T) < outlier_frac
        x[is_out] *= outlier_gain
    if boundary_frac > 0:
        is_bd = rng.random(T) < boundary_frac
        nbd = int(is_bd.sum())
        if nbd:
            f = rng.integers(1, 4, size=nbd).astype(np.float64)
            phi = rng.uniform(0, 2 * np.pi, size=nbd)
            c = np.arange(C, dtype=np.float64)[None, :]
            x[is_bd] = 0.05 * (np.cos(2 * np.pi * f[:, None] * c / C + phi[:, None])
                               + 0.1 * rng.standard_normal(size=(nbd, C)))
    return x.reshape(B, N, C).astype(np.float32)


def weights(rng, O, I, std=0.02):
    return (rng.standard_normal(size=(O, I)) * std).astype(np.float32)


def _case(name, seed, B, N, C, O, bf16, **mix):
    rng = np.random.default_rng(seed)
    x = token_mixture(rng, B, N, C, **mix)
    w = weights(rng, O, C)
    if bf16:
        x = f32_to_bf16_bits(x)
    return LinearCase(name=name, x=x, w=w, x_is_bf16=bf16, meta=dict(seed=seed, **mix))


_MIX_DEFAULT = dict(sigma_log_std=0.5, bg_frac=0.10, bg_nu=3.0, bg_amp=20.0)


def config1(seed=0):
    """Single linear layer: X fp32 [1,256,64], W [64,64]."""
    return _case("cfg1_single_linear_fp32", seed, 1, 256, 64, 64, False, **_MIX_DEFAULT)


def config2(seed=1):
    """Hierarchical-encoder stage-1 MLP fc1: X bf16 [1,9216,64], W [256,64], 1% boundary tokens."""
    return _case("cfg2_stage1_fc1", seed, 1, 9216, 64, 256, True, boundary_frac=0.01, **_MIX_DEFAULT)


def config3(seed=2):
    """Stage-3 qkv projection: X bf16 [16,576,320], 15% Student-t(2.5) x30 tokens, W [960,320]."""
    return _case("cfg3_stage3_qkv", seed, 16, 576, 320, 960, True,
                 sigma_log_std=0.5, bg_frac=0.15, bg_nu=2.5, bg_amp=30.0)


def config4(seed=3, batch=32):
    """ViT-B-style MLP fc1: X bf16 [32,577,768], ln sigma_t ~ N(0,1), 5% tokens x50, W [3072,768]."""
    return _case("cfg4_vitb_fc1", seed, batch, 577, 768, 3072, True,
                 sigma_log_std=1.0, bg_frac=0.0, bg_nu=3.0, bg_amp=1.0,
                 outlier_frac=0.05, outlier_gain=50.0)


# 4-stage encoder at 384x384 input, stride 4: (tokens, channels) per stage, 2 blocks each,
# and per block qkv C->3C, proj C->C, fc1 C->4C, fc2 4C->C in execution order.
SWEEP_STAGES = [(9216, 64), (2304, 128), (576, 320), (144, 512)]


def sweep_shapes(batch=8):
    """[(name, M, I, O)] for the 32 linears of the encoder sweep."""
    out = []
    for s, (tokens, C) in enumerate(SWEEP_STAGES, start=1):
        M = batch * tokens
        for b in range(2):
            for lname, I, O in (("qkv", C, 3 * C), ("proj", C, C), ("fc1", C, 4 * C), ("fc2", 4 * C, C)):
                out.append(("s%d.b%d.%s" % (s, b, lname), M, I, O))
    return out


def config5_layer(layer_index, batch=8):
    """Layer `layer_index` (0..31) of the sweep; its seed is 100 + layer_index."""
    name, M, I, O = sweep_shapes(batch)[layer_index]
    tokens = M // batch
    c = _case("cfg5_" + name, 100 + layer_index, batch, tokens, I, O, True,
              boundary_frac=0.01, **_MIX_DEFAULT)
    return c


def config(idx):
    """Workloads 1..4 by index."""
    return {1: config1, 2: config2, 3: config3, 4: config4}[idx]()


# --- parity-only edge sets (never timed) ------------------------------------------------------

def edge_rows(C=64, seed=7):
    """Rows built to reach the quantizer's corner cases, float32 [R, C]:
    all-zero, constant, +/- largest bf16, ReLU-sparse (more than 7 zeros per group),
    DC offset of 3 sigma (C1 binds at tau=1), ties at the rank-7 magnitude, tiny values
    below the 1e-8 floors, one huge spike per group, alternating signs of equal size."""
    rng = np.random.default_rng(seed)
    rows = []
    rows.append(np.zeros(C))
    rows.append(np.full(C, 0.75))
    rows.append(np.full(C, -3.0))
    big = float(bf16_bits_to_f32(np.array([0x7F7F], np.uint16))[0])
    rows.append(np.where(np.arange(C) % 2 == 0, big, -big))
    r = rng.standard_normal(C)
    rows.append(np.maximum(r, 0.0))
    rows.append(np.maximum(rng.standard_normal(C) - 0.8, 0.0))
    rows.append(rng.standard_normal(C) + 3.0)
    rows.append(0.1 * rng.standard_normal(C) - 5.0)
    t = rng.standard_normal(C)
    t[np.arange(C) % 4 == 1] = 0.125
    t[np.arange(C) % 4 == 2] = -0.125
    rows.append(t)
    rows.append(1e-10 * rng.standard_normal(C))
    rows.append(3e-9 * rng.standard_normal(C))
    s = 0.01 * rng.standard_normal(C)
    s[::32] = 1000.0
    rows.append(s)
    rows.append(np.where(np.arange(C) % 2 == 0, 1.5, -1.5))
    rows.append(rng.standard_t(2.5, size=C) * 30.0)
    rows.append(np.arange(C, dtype=np.float64) - C / 2)
    rows.append(np.ldexp(1.0, -(np.arange(C) % 40) - 100))
    return np.stack(rows).astype(np.float32)


def dc_offset_tokens(M=512, C=96, seed=11):
    """Gaussian tokens riding on a per-token DC offset of 1.5..6 sigma: C1 binds at tau=1."""
    rng = np.random.default_rng(seed)
    sig = np.exp(rng.normal(0, 0.5, size=(M, 1)))
    off = rng.uniform(1.5, 6.0, size=(M, 1)) * sig * rng.choice([-1.0, 1.0], size=(M, 1))
    return (rng.standard_normal((M, C)) * sig + off).astype(np.float32)
