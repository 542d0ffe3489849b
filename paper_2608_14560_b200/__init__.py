"""B200-native fused block-scaled FP8 MoE forward (DeepSeek-V3 layer).

The product is the CUDA library `libmoe_fp8.so` behind the C ABI in
`include/moe_fp8.h`; `binding` marshals arguments to it.  There is no CPU or
PyTorch fallback: without the built library or without a B200 the calls raise.
"""
from . import synthetic  # noqa: F401  (input recipes; no CUDA needed)
from .binding import MoeFp8, MoeFp8Error, load_library  # noqa: F401

__all__ = ["MoeFp8", "MoeFp8Error", "load_library", "synthetic"]
