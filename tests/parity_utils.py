"""Helpers of the GPU parity tests: tensor conversion and the comparison rules.

Comparison rules (written here once, used by every parity test):
  * integer accumulators: bit-exact;
  * 4-bit codes: bit-exact, except that an element whose quotient x/Delta lies within a few
    ulp of a rounding boundary (a half-integer) may differ; the fraction of such elements is
    reported and must stay below 1e-6;
  * group scales: within 1e-6 relative;
  * float32 outputs: |y - y_ref| <= 1e-5 * max(|y_ref|, 1e-3 * rms(y_ref row)); the floor
    keeps the relative test meaningful where terms of opposite sign cancel.
"""
import numpy as np
import torch

import synth_inputs as si


def to_cuda(a: np.ndarray, bf16: bool = False) -> torch.Tensor:
    """numpy -> CUDA tensor; uint16 arrays with bf16=True are reinterpreted as bfloat16."""
    if bf16:
        assert a.dtype == np.uint16
        return torch.from_numpy(a.view(np.int16).copy()).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def unpack_codes(codes: np.ndarray) -> np.ndarray:
    lo = (codes & 0xF).astype(np.int8)
    hi = (codes >> 4).astype(np.int8)
    lo = np.where(lo >= 8, lo - 16, lo).astype(np.int8)
    hi = np.where(hi >= 8, hi - 16, hi).astype(np.int8)
    return np.stack([lo, hi], -1).reshape(codes.shape[0], -1)


def compare_quantizer(x_f32: np.ndarray, g: int, ref: dict, codes: np.ndarray, scale: np.ndarray,
                      code_budget: float = 1e-6):
    """Checks GPU (codes, scale) against the oracle dict.  Returns a small report dict."""
    assert codes.shape == ref["codes"].shape and scale.shape == ref["scale"].shape
    rs = ref["scale"].astype(np.float64)
    rel = np.abs(scale.astype(np.float64) - rs) / rs
    assert rel.max() <= 1e-6, "scale mismatch: max rel %.3e" % rel.max()
    q = unpack_codes(codes)
    bad = q != ref["q"]
    n_bad = int(bad.sum())
    report = dict(n=q.size, code_mismatch=n_bad, scale_max_rel=float(rel.max()),
                  scale_exact_frac=float((scale == ref["scale"]).mean()))
    if n_bad:
        M, Cp = q.shape
        K = Cp // g
        xp = np.zeros((M, Cp), np.float64)
        xp[:, : x_f32.shape[1]] = x_f32
        d = np.repeat(ref["scale"].astype(np.float64), g, axis=1)
        c = np.repeat(ref["clip"].astype(np.float64), g, axis=1)
        r = np.clip(xp, -c, c) / d
        dist = np.abs(np.abs(r - np.floor(r)) - 0.5)          # distance of the quotient from a half-integer
        near = dist <= 8 * 2.0 ** -23 * np.maximum(np.abs(r), 1.0)
        assert (near[bad]).all(), "code mismatch away from a rounding boundary"
        assert (np.abs(q.astype(int) - ref["q"].astype(int))[bad] <= 1).all()
        assert n_bad / q.size < code_budget, "near-boundary mismatch fraction %.3e" % (n_bad / q.size)
    return report


def y_tolerance(y_ref: np.ndarray) -> np.ndarray:
    rms = np.sqrt((y_ref.astype(np.float64) ** 2).mean(axis=-1, keepdims=True))
    return 1e-5 * np.maximum(np.abs(y_ref), 1e-3 * rms)


def compare_y(y: np.ndarray, y_ref_d: np.ndarray, extra_rel: float = 0.0):
    err = np.abs(y.astype(np.float64) - y_ref_d)
    tol = y_tolerance(y_ref_d) + extra_rel * np.abs(y_ref_d)
    worst = float((err / np.maximum(tol, 1e-300)).max())
    assert worst <= 1.0, "output mismatch: worst err/tol = %.3f" % worst
    return worst


def case_tensors(case: si.LinearCase):
    """(x CUDA tensor [M, C], w CUDA tensor [O, I])"""
    x = to_cuda(case.x.reshape(-1, case.C), bf16=case.x_is_bf16)
    w = to_cuda(case.w)
    return x, w
