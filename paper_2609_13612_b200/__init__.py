"""Fused RoPE + masked attention for sm_100a: Python binding over the C-ABI of libattnfuse.

Argument marshalling only: every step of the path runs in the CUDA kernels.  PyTorch supplies
device memory and streams.  There is no CPU fallback: without the compiled library, or without
a CUDA device, the calls raise.
"""
from .binding import (AttnFuseError, BlockMask, RopeSpec, MaskSpec, bwd, bwd_static, decode, device_status, fwd, fwd_blocks, fwd_host, fwd_hybrid, lib, rope,
                      rope_table, version)

__all__ = ["AttnFuseError", "BlockMask", "RopeSpec", "MaskSpec", "bwd", "bwd_static", "decode", "device_status", "fwd", "fwd_blocks", "fwd_host", "fwd_hybrid", "lib",
           "rope", "rope_table", "version"]
