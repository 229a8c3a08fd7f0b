"""ctypes binding of libtdq.so.  Argument marshalling only: every step runs in the library's
CUDA kernels.  torch is used to allocate device memory and to name the current stream."""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtdq.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        "libtdq.so is missing: build it with `python -m paper_2604_16855_b200.build` "
        "(there is no fallback implementation)")
_lib = ctypes.CDLL(LIB_PATH)

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA, ERR_DEVICE_TIMEOUT = range(7)
F32, BF16, F16 = 0, 1, 2
ENABLE_C1, ENABLE_C2, POW2_STEP = 1, 2, 4

# every symbol include/tdq.h declares
EXPORTS = ["tdq_default_act_params", "tdq_quantize_act", "tdq_quantize_weight", "tdq_w4a4_linear",
           "tdq_quant_linear_fused", "tdq_quant_linear_host", "tdq_quantize_act_nchw", "tdq_quantize_act_fixed", "tdq_w4a4_linear_pow2", "tdq_linear_workspace_bytes",
           "tdq_workspace_status", "tdq_status_string", "tdq_kernel_launch_count", "tdq_w4a4_linear_static",
           "tdq_quantize_status", "tdq_selftest_wait_timeout", "tdq_fold_output_affine", "tdq_measure_mma_clocks"]


class ActParams(ctypes.Structure):
    _fields_ = [("group_size", ctypes.c_int32), ("tau", ctypes.c_float), ("zr", ctypes.c_float),
                ("base_percentile", ctypes.c_float), ("flags", ctypes.c_uint32)]


_i64, _i32, _vp, _sz = ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p, ctypes.c_size_t
_pp = ctypes.POINTER(ActParams)
_lib.tdq_default_act_params.argtypes = [_pp]
_lib.tdq_default_act_params.restype = None
_lib.tdq_quantize_act.argtypes = [_vp, ctypes.c_int, _i64, _i64, _i64, _i64, _pp, _vp, _vp, _vp, _vp]
_lib.tdq_quantize_act.restype = ctypes.c_int
_lib.tdq_quantize_act_nchw.argtypes = [_vp, ctypes.c_int, _i64, _i64, _i64, _i64, _pp, _vp, _vp, _vp, _vp]
_lib.tdq_quantize_act_nchw.restype = ctypes.c_int
_lib.tdq_quantize_act_fixed.argtypes = [_vp, ctypes.c_int, _i64, _i64, _i64, _i64, _i32, ctypes.c_float, _vp, _vp, _vp, _vp]
_lib.tdq_quantize_act_fixed.restype = ctypes.c_int
_lib.tdq_quantize_weight.argtypes = [_vp, ctypes.c_int, _i64, _i64, _i32, _vp, _vp, _vp]
_lib.tdq_quantize_weight.restype = ctypes.c_int
_lib.tdq_w4a4_linear.argtypes = [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _i32, _vp, ctypes.c_int, _i64,
                                 _vp, _vp, _sz, _vp]
_lib.tdq_w4a4_linear.restype = ctypes.c_int
_lib.tdq_w4a4_linear_pow2.argtypes = [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _i32, _vp, ctypes.c_int, _i64, _vp, _sz, _vp]
_lib.tdq_w4a4_linear_pow2.restype = ctypes.c_int
_lib.tdq_w4a4_linear_static.argtypes = [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _i32, _vp, ctypes.c_int, _i64,
                                        _i32, _vp]
_lib.tdq_w4a4_linear_static.restype = ctypes.c_int
_lib.tdq_quant_linear_fused.argtypes = [_vp, ctypes.c_int, _i64, _i64, _i64, _i64, _pp, _vp, _vp, _vp, _i64,
                                        _vp, ctypes.c_int, _i64, _vp, _sz, _vp]
_lib.tdq_quant_linear_fused.restype = ctypes.c_int
_lib.tdq_quant_linear_host.argtypes = [_vp, ctypes.c_int, _i64, _i64, _i64, _pp, _vp, _vp, _vp, _i64, _vp,
                                       ctypes.c_int, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.tdq_quant_linear_host.restype = ctypes.c_int
_lib.tdq_linear_workspace_bytes.argtypes = [_i64, _i64, _i64, _i32]
_lib.tdq_linear_workspace_bytes.restype = _sz
_lib.tdq_workspace_status.argtypes = [_vp, _vp, ctypes.POINTER(ctypes.c_uint32)]
_lib.tdq_workspace_status.restype = ctypes.c_int
_lib.tdq_quantize_status.argtypes = [_vp, ctypes.POINTER(ctypes.c_uint32)]
_lib.tdq_quantize_status.restype = ctypes.c_int
_lib.tdq_selftest_wait_timeout.argtypes = [_i32, _i64, _vp, _vp]
_lib.tdq_selftest_wait_timeout.restype = ctypes.c_int
_lib.tdq_fold_output_affine.argtypes = [_vp, _vp, _vp, _vp, _i64, _vp, _vp, _vp]
_lib.tdq_fold_output_affine.restype = ctypes.c_int
_lib.tdq_measure_mma_clocks.argtypes = [_i32, _i32, _vp, _sz, ctypes.POINTER(ctypes.c_double), _vp]
_lib.tdq_measure_mma_clocks.restype = ctypes.c_int
_lib.tdq_status_string.argtypes = [ctypes.c_int]
_lib.tdq_status_string.restype = ctypes.c_char_p
_lib.tdq_kernel_launch_count.argtypes = []
_lib.tdq_kernel_launch_count.restype = ctypes.c_uint64


class TdqError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__("%s: %s (status %d)" % (where, status_string(code), code))


def lib():
    """The loaded ctypes library (for callers that want the raw C ABI)."""
    return _lib


def status_string(code: int) -> str:
    return _lib.tdq_status_string(int(code)).decode()


def kernel_launch_count() -> int:
    return int(_lib.tdq_kernel_launch_count())


def default_act_params() -> ActParams:
    p = ActParams()
    _lib.tdq_default_act_params(ctypes.byref(p))
    return p


def act_params(g=32, tau=1.0, zr=0.2, p=1.0, flags=ENABLE_C1 | ENABLE_C2) -> ActParams:
    return ActParams(int(g), float(tau), float(zr), float(p), int(flags))


def _check(code, where):
    if code != OK:
        raise TdqError(code, where)


def _dtype_id(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float16:
        return F16          # outputs of the linear layer only; the library refuses it elsewhere
    raise TypeError("tdq takes float32, bfloat16 or (for outputs) float16 tensors, got %s" % t.dtype)


def _stream(t: torch.Tensor):
    return ctypes.c_void_p(torch.cuda.current_stream(t.device).cuda_stream)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _need_cuda(*ts):
    for t in ts:
        if t is not None and not t.is_cuda:
            raise ValueError("tdq runs on CUDA tensors only; there is no CPU path")


def quantize_act(x: torch.Tensor, params: ActParams | None = None, *, codes=None, scale=None, offset=None):
    """tdq_quantize_act on x [..., C] (last dim contiguous, rows equally spaced).

    Returns (codes uint8 [M, C_pad/2], scale float32 [M, K])."""
    _need_cuda(x)
    p = params or default_act_params()
    C = x.shape[-1]
    x2 = x.reshape(-1, C)
    if x2.stride(-1) != 1:
        raise ValueError("the channel axis must be contiguous")
    M = x2.shape[0]
    g = p.group_size
    K = (C + g - 1) // g
    if codes is None:
        codes = torch.empty((M, K * g // 2), dtype=torch.uint8, device=x.device)
    if scale is None:
        scale = torch.empty((M, K), dtype=torch.float32, device=x.device)
    if M == 0:          # nothing to do; an empty tensor has no device pointer to pass
        return codes, scale
    stride = x2.stride(0) if M > 1 else C
    _check(_lib.tdq_quantize_act(_ptr(x2), _dtype_id(x2), 1, M, C, stride, ctypes.byref(p), _ptr(codes),
                                 _ptr(scale), _ptr(offset), _stream(x)), "tdq_quantize_act")
    return codes, scale


def quantize_act_fixed(x: torch.Tensor, radius: float, g: int = 32, *, codes=None, scale=None, offset=None):
    """tdq_quantize_act_fixed: the same clip radius in every group.  Returns (codes [M, C/2], scale [M, C/g])."""
    _need_cuda(x, codes, scale, offset)
    C = x.shape[-1]
    x2 = x.reshape(-1, C)
    M = x2.shape[0]
    if codes is None:
        codes = torch.empty((M, C // 2), dtype=torch.uint8, device=x.device)
    if scale is None:
        scale = torch.empty((M, max(C // g, 1)), dtype=torch.float32, device=x.device)
    stride = x2.stride(0) if M > 1 else C
    _check(_lib.tdq_quantize_act_fixed(_ptr(x2), _dtype_id(x2), 1, M, C, stride, g, radius, _ptr(codes), _ptr(scale),
                                       _ptr(offset), _stream(x)), "tdq_quantize_act_fixed")
    return codes, scale


def quantize_act_nchw(x: torch.Tensor, params: ActParams | None = None, *, codes=None, scale=None, offset=None):
    """tdq_quantize_act_nchw on a contiguous CUDA tensor [B, C, H, W].  Returns (codes [B*H*W, C/2], scale [B*H*W, C/32])."""
    _need_cuda(x, codes, scale, offset)
    p = params or default_act_params()
    if x.dim() != 4 or not x.is_contiguous():
        raise ValueError("x must be a contiguous [B, C, H, W] tensor")
    B, C, H, W = x.shape
    M = B * H * W
    if codes is None:
        codes = torch.empty((M, C // 2), dtype=torch.uint8, device=x.device)
    if scale is None:
        scale = torch.empty((M, max(C // 32, 1)), dtype=torch.float32, device=x.device)
    _check(_lib.tdq_quantize_act_nchw(_ptr(x), _dtype_id(x), B, C, H, W, ctypes.byref(p), _ptr(codes), _ptr(scale),
                                      _ptr(offset), _stream(x)), "tdq_quantize_act_nchw")
    return codes, scale


def quantize_weight(w: torch.Tensor, pad_to: int = 32, *, wcodes=None, wscale=None):
    """tdq_quantize_weight on w [O, I] (contiguous).  Returns (wcodes uint8 [O, I_pad/2], wscale [O])."""
    _need_cuda(w)
    w = w.contiguous()
    O, I = w.shape
    I_pad = (I + pad_to - 1) // pad_to * pad_to
    if wcodes is None:
        wcodes = torch.empty((O, I_pad // 2), dtype=torch.uint8, device=w.device)
    if wscale is None:
        wscale = torch.empty((O,), dtype=torch.float32, device=w.device)
    _check(_lib.tdq_quantize_weight(_ptr(w), _dtype_id(w), O, I, pad_to, _ptr(wcodes), _ptr(wscale), _stream(w)),
           "tdq_quantize_weight")
    return wcodes, wscale


def _check_operands(named, y=None):
    """The layout the C ABI assumes but cannot see: dtype, contiguity, one common device; y may have a row pitch
    but its columns must be adjacent.  `named` is a list of (name, tensor or None, dtype).  Returns the device."""
    dev = None
    for name, t, dt in named:
        if t is None:
            continue
        if t.dtype != dt:
            raise TypeError("%s must be %s, got %s" % (name, dt, t.dtype))
        if not t.is_contiguous():
            raise ValueError("%s must be contiguous" % name)
        if dev is None:
            dev = t.device
        elif t.device != dev:
            raise ValueError("%s is on %s, the other operands on %s" % (name, t.device, dev))
    if y is not None:
        if y.dim() != 2 or (y.shape[1] > 1 and y.stride(1) != 1):
            raise ValueError("y must be a matrix whose columns are adjacent in memory")
        if dev is not None and y.device != dev:
            raise ValueError("y is on %s, the operands on %s" % (y.device, dev))
    return dev


def _linear_operands(xcodes, xscale, wcodes, wscale, bias, y, workspace=None, acc_debug=None):
    return _check_operands([("xcodes", xcodes, torch.uint8), ("xscale", xscale, torch.float32), ("wcodes", wcodes, torch.uint8),
                            ("wscale", wscale, torch.float32), ("bias", bias, torch.float32),
                            ("workspace", workspace, torch.uint8), ("acc_debug", acc_debug, torch.int32)], y)


def linear_workspace(M, I_pad, O, g, device) -> torch.Tensor:
    n = int(_lib.tdq_linear_workspace_bytes(M, I_pad, O, g))
    return torch.zeros((n,), dtype=torch.uint8, device=device)


def w4a4_linear(xcodes, xscale, wcodes, wscale, bias=None, *, g=32, out_dtype=torch.float32, y=None,
                acc_debug=None, workspace=None):
    """tdq_w4a4_linear.  Returns y [M, O]."""
    _need_cuda(xcodes, xscale, wcodes, wscale, bias)
    M, half = xcodes.shape
    I_pad = half * 2
    O = wcodes.shape[0]
    if y is None:
        y = torch.empty((M, O), dtype=out_dtype, device=xcodes.device)
    if workspace is None:
        workspace = linear_workspace(M, I_pad, O, g, xcodes.device)
    dev = _linear_operands(xcodes, xscale, wcodes, wscale, bias, y, workspace, acc_debug)
    with torch.cuda.device(dev):        # the library works on the current device
        _check(_lib.tdq_w4a4_linear(_ptr(xcodes), _ptr(xscale), _ptr(wcodes), _ptr(wscale), _ptr(bias), M, I_pad, O, g,
                                    _ptr(y), _dtype_id(y), y.stride(0) if M > 0 else O, _ptr(acc_debug),
                                    _ptr(workspace), workspace.numel(), _stream(xcodes)), "tdq_w4a4_linear")
    return y


def w4a4_linear_pow2(xcodes, xscale, wcodes, wscale, bias=None, *, g=32, out_dtype=torch.float32, y=None, workspace=None):
    """tdq_w4a4_linear_pow2: the linear layer for power-of-two activation steps.  Returns y [M, O]."""
    _need_cuda(xcodes, xscale, wcodes, wscale, bias)
    M, half = xcodes.shape
    I_pad = half * 2
    O = wcodes.shape[0]
    if y is None:
        y = torch.empty((M, O), dtype=out_dtype, device=xcodes.device)
    if workspace is None:
        workspace = linear_workspace(M, I_pad, O, g, xcodes.device)
    dev = _linear_operands(xcodes, xscale, wcodes, wscale, bias, y, workspace)
    with torch.cuda.device(dev):
        _check(_lib.tdq_w4a4_linear_pow2(_ptr(xcodes), _ptr(xscale), _ptr(wcodes), _ptr(wscale), _ptr(bias), M, I_pad, O, g,
                                         _ptr(y), _dtype_id(y), y.stride(0) if M > 0 else O, _ptr(workspace),
                                         workspace.numel(), _stream(xcodes)), "tdq_w4a4_linear_pow2")
    return y


LINEAR_STATIC_BYTES = 8 << 20   # TDQ_LINEAR_STATIC_BYTES of the header


def w4a4_linear_static(xcodes, xscale, wcodes, wscale, bias=None, *, g=32, y, wait=True):
    """tdq_w4a4_linear_static: the linear layer for callers that may not allocate device memory.

    The scratch space is a fixed array inside the library, so this wrapper allocates nothing
    either: the caller passes the output tensor y [M, O].  Returns y."""
    _need_cuda(xcodes, xscale, wcodes, wscale, bias, y)
    M, half = xcodes.shape
    O = wcodes.shape[0]
    dev = _linear_operands(xcodes, xscale, wcodes, wscale, bias, y)
    with torch.cuda.device(dev):        # the scratch array is looked up on the current device
        _check(_lib.tdq_w4a4_linear_static(_ptr(xcodes), _ptr(xscale), _ptr(wcodes), _ptr(wscale), _ptr(bias), M, half * 2,
                                           O, g, _ptr(y), _dtype_id(y), y.stride(0) if M > 0 else O, 1 if wait else 0,
                                           _stream(xcodes)), "tdq_w4a4_linear_static")
    return y


def quant_linear_fused(x, wcodes, wscale, bias=None, params: ActParams | None = None, *,
                       out_dtype=torch.float32, y=None, workspace=None):
    """tdq_quant_linear_fused: quantizer as the linear layer's A-operand producer.  Returns y [M, O]."""
    _need_cuda(x, wcodes, wscale, bias)
    p = params or default_act_params()
    C = x.shape[-1]
    x2 = x.reshape(-1, C)
    M = x2.shape[0]
    O = wcodes.shape[0]
    if y is None:
        y = torch.empty((M, O), dtype=out_dtype, device=x.device)
    if workspace is None:
        workspace = linear_workspace(M, wcodes.shape[1] * 2, O, p.group_size, x.device)
    stride = x2.stride(0) if M > 1 else C
    if x2.dim() != 2 or (C > 1 and x2.stride(1) != 1):
        raise ValueError("the channels of x must be adjacent in memory")
    dev = _check_operands([("wcodes", wcodes, torch.uint8), ("wscale", wscale, torch.float32), ("bias", bias, torch.float32),
                           ("workspace", workspace, torch.uint8)], y)
    if x2.device != dev:
        raise ValueError("x is on %s, the weights on %s" % (x2.device, dev))
    with torch.cuda.device(dev):
        _check(_lib.tdq_quant_linear_fused(_ptr(x2), _dtype_id(x2), 1, M, C, stride, ctypes.byref(p), _ptr(wcodes),
                                           _ptr(wscale), _ptr(bias), O, _ptr(y), _dtype_id(y), y.stride(0),
                                           _ptr(workspace), workspace.numel(), _stream(x)), "tdq_quant_linear_fused")
    return y


def quant_linear_host(x_host: torch.Tensor, wcodes, wscale, bias=None, params: ActParams | None = None, *,
                      out_dtype=torch.float32, y_host=None, device="cuda"):
    """tdq_quant_linear_host: x_host [M, C] (CPU, ideally pinned) in, y_host [M, O] (CPU) out.  The device buffers
    the call needs are allocated here.  Returns (y_host, workspace); synchronise the current stream before reading."""
    _need_cuda(wcodes, wscale, bias)
    p = params or default_act_params()
    M, C = x_host.shape
    O = wcodes.shape[0]
    g = p.group_size
    I_pad = (C + g - 1) // g * g
    dev = wcodes.device
    x_dev = torch.empty((M, C), dtype=x_host.dtype, device=dev)
    codes = torch.empty((M, I_pad // 2), dtype=torch.uint8, device=dev)
    scale = torch.empty((M, I_pad // g), dtype=torch.float32, device=dev)
    y_dev = torch.empty((M, O), dtype=out_dtype, device=dev)
    if y_host is None:
        y_host = torch.empty((M, O), dtype=out_dtype).pin_memory()
    workspace = linear_workspace(M, I_pad, O, g, dev)
    _check(_lib.tdq_quant_linear_host(_ptr(x_host), _dtype_id(x_host), 1, M, C, ctypes.byref(p), _ptr(wcodes), _ptr(wscale),
                                      _ptr(bias), O, _ptr(y_host), _dtype_id(y_host), _ptr(x_dev), _ptr(codes), _ptr(scale),
                                      _ptr(y_dev), _ptr(workspace), workspace.numel(), _stream(wcodes)),
           "tdq_quant_linear_host")
    return y_host, (workspace, x_dev, codes, scale, y_dev)


def workspace_status(workspace: torch.Tensor):
    """(status, detail word) left by the last linear call that used this workspace; synchronises."""
    detail = ctypes.c_uint32(0)
    st = _lib.tdq_workspace_status(_ptr(workspace), _stream(workspace), ctypes.byref(detail))
    return int(st), int(detail.value)


def quantize_status(device=None):
    """(status, detail) of the quantizer kernels' bounded waits on the current stream's device; clears the word."""
    detail = ctypes.c_uint32(0)
    st = _lib.tdq_quantize_status(ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream), ctypes.byref(detail))
    return st, detail.value


def selftest_wait_timeout(which: int, limit_cycles: int, workspace: torch.Tensor | None = None):
    """Makes one bounded wait run out (see tdq.h); the status is read with workspace_status / quantize_status."""
    ws = ctypes.c_void_p(workspace.data_ptr()) if workspace is not None else None
    dev = workspace.device if workspace is not None else None
    _check(_lib.tdq_selftest_wait_timeout(which, limit_cycles, ws, ctypes.c_void_p(torch.cuda.current_stream(dev).cuda_stream)),
           "tdq_selftest_wait_timeout")


def fold_output_affine(wscale, bias, out_mul, out_add=None):
    """tdq_fold_output_affine: (wscale', bias') such that the linear layer computes out_mul * y + out_add."""
    _need_cuda(wscale, bias, out_mul, out_add)
    dev = _check_operands([("wscale", wscale, torch.float32), ("bias", bias, torch.float32), ("out_mul", out_mul, torch.float32),
                           ("out_add", out_add, torch.float32)])
    O = wscale.shape[0]
    ws2, b2 = torch.empty_like(wscale), torch.empty_like(wscale)
    with torch.cuda.device(dev):
        _check(_lib.tdq_fold_output_affine(_ptr(wscale), _ptr(bias), _ptr(out_mul), _ptr(out_add), O, _ptr(ws2), _ptr(b2),
                                           _stream(wscale)), "tdq_fold_output_affine")
    return ws2, b2


def measure_mma_clocks(integer_kind: bool, n_mma: int = 8192, device="cuda") -> float:
    """tdq_measure_mma_clocks: clocks per 128 x 128 x 32 tensor-core instruction on the slowest SM of the device."""
    dev = torch.device(device)
    scratch = torch.zeros((16 * 1024,), dtype=torch.uint8, device=dev)
    out = ctypes.c_double(0.0)
    with torch.cuda.device(dev):
        _check(_lib.tdq_measure_mma_clocks(1 if integer_kind else 0, n_mma, _ptr(scratch), scratch.numel(), ctypes.byref(out),
                                           ctypes.c_void_p(torch.cuda.current_stream(dev).cuda_stream)), "tdq_measure_mma_clocks")
    return float(out.value)
