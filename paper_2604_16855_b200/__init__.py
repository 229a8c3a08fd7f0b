"""B200-native COD-TDQ hot path: token-group dual-constraint activation quantizer and W4A4
linear layer, as a C-ABI CUDA library (``libtdq.so``) with a thin ctypes binding.

    from paper_2604_16855_b200 import tdq
    codes, scale = tdq.quantize_act(x)                     # x: CUDA tensor [B, N, C], fp32 or bf16
    wcodes, wscale = tdq.quantize_weight(w)
    y = tdq.w4a4_linear(codes, scale, wcodes, wscale)

Importing the package loads the library and fails if it has not been built
(``python -m paper_2604_16855_b200.build``).  There is no CPU or PyTorch fallback.
"""
from . import binding as tdq  # noqa: F401

__all__ = ["tdq"]
