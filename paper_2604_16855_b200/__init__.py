"""B200-native COD-TDQ hot path: token-group dual-constraint activation quantizer and W4A4
linear layer, as a C-ABI CUDA library (``libtdq.so``) with a thin ctypes binding.

    from paper_2604_16855_b200 import tdq
    codes, scale = tdq.quantize_act(x)                     # x: CUDA tensor [B, N, C], fp32 or bf16
    wcodes, wscale = tdq.quantize_weight(w)
    y = tdq.w4a4_linear(codes, scale, wcodes, wscale)

``tdq`` (the binding module) is loaded on first access and fails if the library has not been
built (``python -m paper_2604_16855_b200.build``).  There is no CPU or PyTorch fallback.  The
``build`` submodule imports without the library, so that it can create it.
"""
import importlib

__all__ = ["tdq"]


def __getattr__(name):
    if name == "tdq":
        mod = importlib.import_module(".binding", __name__)
        globals()["tdq"] = mod
        return mod
    raise AttributeError("module %r has no attribute %r" % (__name__, name))
