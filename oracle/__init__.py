"""ctypes front end of the CPU oracle (``tdq_oracle.c``).

Test infrastructure only: the tests, the smoke check and the benchmark's CPU
baseline may import this module; the CUDA library and its Python binding never
do.  Arrays are numpy, on the host.  The shared object is compiled with gcc on
first use and kept next to the source.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tdq_oracle.c")
_SO = os.path.join(_HERE, "libtdq_oracle.so")
_lock = threading.Lock()
_lib = None

F32 = 0
BF16 = 1
ENABLE_C1 = 1
ENABLE_C2 = 2
POW2_STEP = 4


def build(force: bool = False) -> str:
    """Compile the oracle with gcc; returns the path of the shared object."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            i64, i32, u32, f32, vp = (ctypes.c_int64, ctypes.c_int32, ctypes.c_uint32,
                                      ctypes.c_float, ctypes.c_void_p)
            lib.tdq_oracle_rank.argtypes = [f32, i32]
            lib.tdq_oracle_rank.restype = i32
            lib.tdq_oracle_quantize_act.argtypes = [vp, ctypes.c_int, i64, i64, i64, i32, f32, f32,
                                                    f32, u32, vp, vp, vp, vp, vp]
            lib.tdq_oracle_quantize_act.restype = ctypes.c_int
            lib.tdq_oracle_quantize_act_fixed.argtypes = [vp, ctypes.c_int, i64, i64, i64, i32, f32, vp, vp, vp]
            lib.tdq_oracle_quantize_act_fixed.restype = ctypes.c_int
            lib.tdq_oracle_quantize_weight.argtypes = [vp, ctypes.c_int, i64, i64, i32, vp, vp, vp]
            lib.tdq_oracle_quantize_weight.restype = ctypes.c_int
            lib.tdq_oracle_w4a4_linear.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, i32, vp, vp, vp, vp]
            lib.tdq_oracle_w4a4_linear.restype = ctypes.c_int
            lib.tdq_oracle_num_threads.restype = ctypes.c_int
            _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _as_input(x):
    """(contiguous array, dtype id): float32 arrays are F32, uint16 arrays hold bf16 bits."""
    x = np.ascontiguousarray(x)
    if x.dtype == np.float32:
        return x, F32
    if x.dtype == np.uint16:
        return x, BF16
    raise TypeError("oracle inputs are float32 or uint16 (bf16 bit patterns), got %s" % x.dtype)


def rank(frac: float, g: int) -> int:
    """1-indexed order-statistic rank ceil(frac * g) (Supp. S2.2)."""
    return int(_load().tdq_oracle_rank(float(np.float32(frac)), int(g)))


def num_threads() -> int:
    return int(_load().tdq_oracle_num_threads())


def quantize_act(x, g=32, tau=1.0, zr=0.2, p=1.0, flags=ENABLE_C1 | ENABLE_C2, C=None):
    """Algorithm S1 steps 1-9 on x of shape [..., C].

    With C given, x is [M, row_stride] and only the first C channels of each row are read.

    Returns a dict: q int8 [M, C_pad], codes uint8 [M, C_pad/2], scale float32 [M, K],
    clip float32 [M, K], active uint8 [M, K] (0 base, 1 C1, 2 C2).
    """
    x, dt = _as_input(x)
    row_stride = x.shape[-1]
    C = row_stride if C is None else int(C)
    M = int(np.prod(x.shape[:-1])) if x.ndim > 1 else 1
    K = (C + g - 1) // g
    C_pad = K * g
    out = dict(q=np.empty((M, C_pad), np.int8), codes=np.empty((M, C_pad // 2), np.uint8),
               scale=np.empty((M, K), np.float32), clip=np.empty((M, K), np.float32),
               active=np.empty((M, K), np.uint8))
    rc = _load().tdq_oracle_quantize_act(_ptr(x), dt, M, C, row_stride,
                                         g, tau, zr, p, flags, _ptr(out["q"]), _ptr(out["codes"]),
                                         _ptr(out["scale"]), _ptr(out["clip"]), _ptr(out["active"]))
    if rc != 0:
        raise ValueError("tdq_oracle_quantize_act rejected its arguments")
    return out


def quantize_act_fixed(x, radius, g=32, C=None):
    """The fixed-radius control: steps 5-9 of Algorithm S1 with the same given clip radius in every group.
    Returns a dict: q int8 [M, C_pad], codes uint8 [M, C_pad/2], scale float32 [M, K]."""
    x, dt = _as_input(x)
    row_stride = x.shape[-1]
    C = row_stride if C is None else int(C)
    M = int(np.prod(x.shape[:-1])) if x.ndim > 1 else 1
    K = (C + g - 1) // g
    C_pad = K * g
    out = dict(q=np.empty((M, C_pad), np.int8), codes=np.empty((M, C_pad // 2), np.uint8),
               scale=np.empty((M, K), np.float32))
    rc = _load().tdq_oracle_quantize_act_fixed(_ptr(x), dt, M, C, row_stride, g, float(radius),
                                               _ptr(out["q"]), _ptr(out["codes"]), _ptr(out["scale"]))
    if rc != 0:
        raise ValueError("tdq_oracle_quantize_act_fixed rejected its arguments")
    return out


def quantize_act_nchw(x, **kw):
    """The 4-D branch of Supp. S1.1: a feature map [B, C, H, W] is laid out as tokens [B, H*W, C] (a plain
    transpose), then quantized along C by quantize_act.  Outputs are token-major: [B*H*W, ...]."""
    x = np.asarray(x)
    if x.ndim != 4:
        raise ValueError("x must be [B, C, H, W]")
    B, C, H, W = x.shape
    tokens = np.ascontiguousarray(np.transpose(x, (0, 2, 3, 1))).reshape(B * H * W, C)
    return quantize_act(tokens, **kw)


def quantize_weight(w, pad_to=32):
    """Eq. 4 with absmax scales. Returns dict q int8 [O, I_pad], codes uint8, scale float32 [O]."""
    w, dt = _as_input(w)
    O, I = w.shape
    I_pad = (I + pad_to - 1) // pad_to * pad_to
    out = dict(q=np.empty((O, I_pad), np.int8), codes=np.empty((O, I_pad // 2), np.uint8),
               scale=np.empty((O,), np.float32))
    rc = _load().tdq_oracle_quantize_weight(_ptr(w), dt, O, I, pad_to, _ptr(out["q"]),
                                            _ptr(out["codes"]), _ptr(out["scale"]))
    if rc != 0:
        raise ValueError("tdq_oracle_quantize_weight rejected its arguments")
    return out


def w4a4_linear(xcodes, xscale, wcodes, wscale, bias=None, g=32, want_acc=False):
    """Algorithm S1 step 10 as an integer contraction plus scaling.

    Returns dict y float32 [M, O], y_d float64 [M, O], t_abs float64 [M, O] (size of the summed
    terms, s_o * sum_k Delta_k |acc_k|) and, when asked, acc int32 [M, O, K].
    """
    xcodes = np.ascontiguousarray(xcodes, np.uint8)
    wcodes = np.ascontiguousarray(wcodes, np.uint8)
    xscale = np.ascontiguousarray(xscale, np.float32)
    wscale = np.ascontiguousarray(wscale, np.float32)
    bias = None if bias is None else np.ascontiguousarray(bias, np.float32)
    M, half = xcodes.shape
    I_pad = half * 2
    O = wcodes.shape[0]
    K = I_pad // g
    assert wcodes.shape[1] == half and xscale.shape == (M, K) and wscale.shape == (O,)
    out = dict(y=np.empty((M, O), np.float32), y_d=np.empty((M, O), np.float64),
               t_abs=np.empty((M, O), np.float64))
    acc = np.empty((M, O, K), np.int32) if want_acc else None
    rc = _load().tdq_oracle_w4a4_linear(_ptr(xcodes), _ptr(xscale), _ptr(wcodes), _ptr(wscale),
                                        _ptr(bias), M, I_pad, O, g, _ptr(out["y"]), _ptr(out["y_d"]),
                                        _ptr(acc), _ptr(out["t_abs"]))
    if rc != 0:
        raise ValueError("tdq_oracle_w4a4_linear rejected its arguments")
    if want_acc:
        out["acc"] = acc
    return out


def output_affine(ref, out_mul, out_add=None, bias=None):
    """The affine mode of the auxiliary Linear I/O correction (Supp. S1.1): y' = a_o * y + b_o per output channel,
    applied in binary64 to the dict w4a4_linear returns (y_d, t_abs; y is y_d rounded to binary32).  t_abs, the
    diagnostic size of the summed terms, is scaled by |a_o|; when the layer's bias is passed, |a_o bias_o| and
    |b_o| are added to it (the constants a folded evaluation rounds)."""
    a = np.asarray(out_mul, np.float64)[None, :]
    b = 0.0 if out_add is None else np.asarray(out_add, np.float64)[None, :]
    y_d = a * ref["y_d"] + b
    t_abs = np.abs(a) * ref["t_abs"]
    if bias is not None:
        t_abs = t_abs + np.abs(a * np.asarray(bias, np.float64)[None, :])
        t_abs = t_abs + np.abs(b)
    return dict(y=y_d.astype(np.float32), y_d=y_d, t_abs=t_abs)
