"""Helpers of the GPU parity tests: tensor conversion and the comparison rules.

Comparison rules (written here once, used by every parity test):
  * integer accumulators: bit-exact;
  * 4-bit codes: bit-exact, except that an element whose quotient x/Delta lies within a few
    ulp of a rounding boundary (a half-integer) may differ; the fraction of such elements is
    reported and must stay below 1e-6;
  * group scales: within 1e-6 relative;
  * float32 outputs: within 1e-5 relative, or within the binary32 rounding bound of the
    sum's own terms where they cancel (see compare_y).
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


def compare_y(y: np.ndarray, ref: dict, n_groups: int, out_eps: float = 0.0):
    """|y - y_ref| <= max(1e-5 |y_ref|, (K+2) 2^-24 T) + out_eps |y_ref|, T = s_o sum_k Delta_k |acc_k|.

    The second term is the binary32 rounding bound of the K-term sum itself: where the terms
    cancel, |y_ref| can be arbitrarily smaller than T and no float32 evaluation of the sum can
    be accurate to 1e-5 of |y_ref|.  Returns (worst err/tol, fraction passing the plain
    1e-5 relative rule)."""
    y_ref = ref["y_d"]
    err = np.abs(y.astype(np.float64) - y_ref)
    tol = np.maximum(1e-5 * np.abs(y_ref), (n_groups + 2) * 2.0 ** -24 * ref["t_abs"]) + out_eps * np.abs(y_ref)
    worst = float((err / np.maximum(tol, 1e-300)).max())
    assert worst <= 1.0, "output mismatch: worst err/tol = %.3f" % worst
    strict = float((err <= 1e-5 * np.abs(y_ref) + 1e-300).mean())
    return worst, strict


def case_tensors(case: si.LinearCase):
    """(x CUDA tensor [M, C], w CUDA tensor [O, I])"""
    x = to_cuda(case.x.reshape(-1, case.C), bf16=case.x_is_bf16)
    w = to_cuda(case.w)
    return x, w
