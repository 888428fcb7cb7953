"""B200-native compression step of LIEC-SGD (Algorithm 1): thin Python binding over the C ABI.

``liec`` holds the ctypes declarations and a small ``Context`` helper; every numeric step
runs in the CUDA library ``libliec.so`` built by ``paper_2402_11857_b200.build``.
"""
from . import liec
from .liec import (Context, LiecError, COMP_IDENTITY, COMP_SCALED_SIGN, COMP_TOPK, F32, BF16,
                   load_library, workspace_bytes, down_message_bytes)

__all__ = ["liec", "Context", "LiecError", "COMP_IDENTITY", "COMP_SCALED_SIGN", "COMP_TOPK",
           "F32", "BF16", "load_library", "workspace_bytes", "down_message_bytes"]
