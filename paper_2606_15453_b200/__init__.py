"""B200-native decode-time MoE layer step with the ST-MoE expert predictor.

Thin Python access to the C-ABI library (libstmoe.so, built from csrc/ by build.py).
All computation runs in the library's CUDA kernels; this package only marshals
arguments.  There is no CPU path: importing works anywhere, every call needs a GPU.
"""
from .binding import (Stack, StmoeError, expert_image_bytes, lib, moe_ffn,  # noqa: F401
                      moe_ffn_scratch_bytes, moe_ffn_static, expert_ffn_dense, router_topk, DTYPE, MODE, FLAG_RENORM_TOPK, FLAG_NO_PERSISTENT, FLAG_NO_DENSE, FLAG_NO_FUSED)
from .build import build  # noqa: F401
