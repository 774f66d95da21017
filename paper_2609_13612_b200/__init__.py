"""Fused RoPE + masked attention for sm_100a: Python binding over the C-ABI of libattnfuse.

Argument marshalling only: every step of the path runs in the CUDA kernels.  PyTorch supplies
device memory and streams.  There is no CPU fallback: without the compiled library, or without
a CUDA device, the calls raise.
"""
from .binding import (AttnFuseError, BlockMask, RopeSpec, MaskSpec, bwd, bwd_static, bwd_variant, bwd_workspace_bytes, decode, decode_workspace, device_status, fwd, fwd_blocks, fwd_fp8, fwd_host, fwd_hybrid, fwd_variant, get_option, lib, option, rope,
                      rope_table, selftest_wait_timeout, set_option, stream_status, version)
from . import binding as _b

OPT_FWD_QTILES, OPT_FWD_PAIR_HEADS = _b.OPT_FWD_QTILES, _b.OPT_FWD_PAIR_HEADS
OPT_FWD_KEYS_BF16, OPT_BS_ROWPAIR = _b.OPT_FWD_KEYS_BF16, _b.OPT_BS_ROWPAIR
OPT_BWD_ONEPASS, OPT_FWD_ALIBI_MMA = _b.OPT_BWD_ONEPASS, _b.OPT_FWD_ALIBI_MMA

__all__ = ["AttnFuseError", "BlockMask", "RopeSpec", "MaskSpec", "bwd", "bwd_static", "bwd_variant", "bwd_workspace_bytes", "decode", "decode_workspace", "device_status", "fwd", "fwd_blocks", "fwd_fp8", "fwd_host", "fwd_hybrid", "fwd_variant", "get_option", "lib",
           "option", "rope", "rope_table", "selftest_wait_timeout", "set_option", "stream_status", "version"]
