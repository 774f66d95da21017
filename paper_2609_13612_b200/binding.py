"""ctypes binding with the same names as the C entry points (see include/attnfuse.h)."""
from __future__ import annotations

import ctypes
import dataclasses
import os
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libattnfuse.so")

AF_BF16, AF_F32 = 0, 1


class AttnFuseError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__("attnfuse error %d: %s" % (code, msg))
        self.code = code


class _Shape(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int), ("Hq", ctypes.c_int), ("Hkv", ctypes.c_int), ("S", ctypes.c_int),
                ("D", ctypes.c_int)]


class _Strides(ctypes.Structure):
    _fields_ = [("b", ctypes.c_int64), ("h", ctypes.c_int64), ("s", ctypes.c_int64)]


class _Blocks(ctypes.Structure):
    _fields_ = [("block", ctypes.c_int), ("row_ptr", ctypes.c_void_p), ("col_idx", ctypes.c_void_p),
                ("col_ptr", ctypes.c_void_p), ("row_idx", ctypes.c_void_p), ("row_order", ctypes.c_void_p),
                ("col_order", ctypes.c_void_p), ("pair_ptr", ctypes.c_void_p), ("pair_idx", ctypes.c_void_p),
                ("pair_order", ctypes.c_void_p)]


class _Variant(ctypes.Structure):
    pass


class _Rope(ctypes.Structure):
    _fields_ = [("theta", ctypes.c_float), ("rotary_dim", ctypes.c_int), ("pos_offset", ctypes.c_int)]


class _Mask(ctypes.Structure):
    _fields_ = [("causal", ctypes.c_int), ("window", ctypes.c_int), ("alibi_slopes", ctypes.c_void_p)]


_Variant._fields_ = [("rope", _Rope), ("rope_table", ctypes.c_void_p), ("mask", _Mask), ("bias", ctypes.c_void_p),
                     ("bias_B", ctypes.c_int), ("bias_H", ctypes.c_int), ("normaliser", ctypes.c_int),
                     ("blocks", ctypes.POINTER(_Blocks))]


@dataclasses.dataclass(frozen=True)
class RopeSpec:
    theta: float = 10000.0
    rotary_dim: int = 0
    pos_offset: int = 0


@dataclasses.dataclass
class MaskSpec:
    causal: bool = True
    window: int = -1
    alibi_slopes: Optional[torch.Tensor] = None  # fp32 [Hq] on the device


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise AttnFuseError(-1, "libattnfuse.so is not built; run `python -m paper_2609_13612_b200.build`")
        L = ctypes.CDLL(_LIB_PATH)
        vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        P = ctypes.POINTER
        L.attnfuse_version.restype = i
        L.attnfuse_strerror.restype = ctypes.c_char_p
        L.attnfuse_strerror.argtypes = [i]
        L.attnfuse_set_option.restype = i
        L.attnfuse_set_option.argtypes = [i, i]
        L.attnfuse_get_option.restype = i
        L.attnfuse_get_option.argtypes = [i]
        L.attnfuse_device_status.restype = i
        L.attnfuse_device_status.argtypes = [P(ctypes.c_uint)]
        L.attnfuse_stream_status.restype = i
        L.attnfuse_stream_status.argtypes = [vp, P(ctypes.c_uint)]
        L.attnfuse_selftest_wait_timeout.restype = i
        L.attnfuse_selftest_wait_timeout.argtypes = [ctypes.c_uint, vp]
        L.attnfuse_rope_table_bytes.restype = sz
        L.attnfuse_rope_table_bytes.argtypes = [i, i]
        L.attnfuse_rope_table.restype = i
        L.attnfuse_rope_table.argtypes = [P(_Rope), i, vp, vp]
        L.attnfuse_rope.restype = i
        L.attnfuse_rope.argtypes = [P(_Shape), i, vp, vp, P(_Rope), vp, i, vp]
        L.attnfuse_fwd.restype = i
        L.attnfuse_fwd.argtypes = [P(_Shape), vp, vp, vp, P(_Strides), P(_Strides), P(_Rope), vp, P(_Mask), i, f,
                                   vp, i, vp, vp]
        L.attnfuse_fwd_fp8.restype = i
        L.attnfuse_fwd_fp8.argtypes = [P(_Shape), vp, vp, vp, P(_Mask), i, f, f, f, f, vp, i, vp, vp]
        L.attnfuse_fwd_variant.restype = i
        L.attnfuse_fwd_variant.argtypes = [P(_Shape), vp, vp, vp, P(_Strides), P(_Strides), P(_Variant), i, f, vp, i, vp, vp]
        L.attnfuse_fwd_hybrid_workspace_bytes.restype = sz
        L.attnfuse_fwd_hybrid_workspace_bytes.argtypes = [P(_Shape)]
        L.attnfuse_fwd_hybrid.restype = i
        L.attnfuse_fwd_hybrid.argtypes = [P(_Shape), vp, vp, vp, P(_Strides), P(_Strides), P(_Rope), vp, P(_Mask), i, f,
                                          vp, i, vp, vp, sz, vp]
        L.attnfuse_fwd_host_staging_bytes.restype = sz
        L.attnfuse_fwd_host_staging_bytes.argtypes = [P(_Shape)]
        L.attnfuse_fwd_host.restype = i
        L.attnfuse_fwd_host.argtypes = [P(_Shape), vp, vp, vp, P(_Rope), vp, P(_Mask), i, f, vp, vp, vp, sz, vp]
        L.attnfuse_bwd_workspace_bytes.restype = sz
        L.attnfuse_bwd_workspace_bytes.argtypes = [P(_Shape)]
        L.attnfuse_bwd_onepass_workspace_bytes.restype = sz
        L.attnfuse_bwd_onepass_workspace_bytes.argtypes = [P(_Shape)]
        L.attnfuse_bwd.restype = i
        L.attnfuse_bwd.argtypes = [P(_Shape), vp, vp, vp, vp, vp, vp, P(_Strides), P(_Strides), P(_Rope), vp,
                                   P(_Mask), i, f, vp, i, vp, vp, i, vp, sz, vp]
        L.attnfuse_bwd_variant.restype = i
        L.attnfuse_bwd_variant.argtypes = [P(_Shape), vp, vp, vp, vp, vp, vp, P(_Strides), P(_Strides), P(_Variant), i, f,
                                           vp, i, vp, vp, i, vp, sz, vp]
        L.attnfuse_fwd_blocks.restype = i
        L.attnfuse_fwd_blocks.argtypes = [P(_Shape), vp, vp, vp, P(_Strides), P(_Strides), P(_Rope), vp, P(_Mask), i, f,
                                          P(_Blocks), vp, i, vp, vp]
        L.attnfuse_bwd_blocks.restype = i
        L.attnfuse_bwd_blocks.argtypes = [P(_Shape), vp, vp, vp, vp, vp, vp, P(_Strides), P(_Strides), P(_Rope), vp,
                                          P(_Mask), i, f, P(_Blocks), vp, i, vp, vp, i, vp, sz, vp]
        L.attnfuse_decode_splits.restype = i
        L.attnfuse_decode_splits.argtypes = [P(_Shape)]
        L.attnfuse_decode_workspace_bytes.restype = sz
        L.attnfuse_decode_workspace_bytes.argtypes = [P(_Shape), i]
        L.attnfuse_decode_workspace_init.restype = i
        L.attnfuse_decode_workspace_init.argtypes = [vp, sz, vp]
        L.attnfuse_decode.restype = i
        L.attnfuse_decode.argtypes = [P(_Shape), vp, vp, vp, P(_Strides), P(_Mask), i, f, vp, vp, i, vp, sz, vp]
        L.attnfuse_bwd_static.restype = i
        L.attnfuse_bwd_static.argtypes = [P(_Shape), vp, vp, vp, vp, vp, vp, P(_Strides), P(_Strides), P(_Rope), vp,
                                          P(_Mask), i, f, vp, i, vp, vp, i, vp]
        _lib = L
    return _lib


def _check(code: int):
    if code != 0:
        raise AttnFuseError(code, lib().attnfuse_strerror(code).decode())


def version() -> int:
    return lib().attnfuse_version()


# af_option values (include/attnfuse.h)
OPT_FWD_QTILES, OPT_FWD_PAIR_HEADS, OPT_FWD_KEYS_BF16, OPT_BS_ROWPAIR, OPT_BWD_ONEPASS, OPT_FWD_ALIBI_MMA = range(6)


def set_option(option: int, value: int) -> None:
    _check(lib().attnfuse_set_option(option, value))


def get_option(option: int) -> int:
    return lib().attnfuse_get_option(option)


class option:
    """Context manager: a tuning option set for the duration of a block, then restored."""

    def __init__(self, opt: int, value: int):
        self.opt, self.value = opt, value

    def __enter__(self):
        self.old = get_option(self.opt)
        set_option(self.opt, self.value)
        return self

    def __exit__(self, *exc):
        set_option(self.opt, self.old)
        return False


def device_status() -> Tuple[int, int]:
    d = ctypes.c_uint(0)
    code = lib().attnfuse_device_status(ctypes.byref(d))
    return code, d.value


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def stream_status() -> Tuple[int, int]:
    """Status word read in order on the current stream (synchronises that stream only)."""
    d = ctypes.c_uint(0)
    code = lib().attnfuse_stream_status(_stream(), ctypes.byref(d))
    return code, d.value


def selftest_wait_timeout(limit_cycles: int = 2_000_000) -> None:
    """Launch the self-test CTA whose bounded wait runs out after `limit_cycles` SM clocks."""
    _check(lib().attnfuse_selftest_wait_timeout(limit_cycles, _stream()))


def _need_cuda(*ts):
    for t in ts:
        if t is not None and not t.is_cuda:
            raise AttnFuseError(-2, "tensor is not on a CUDA device (there is no CPU path)")


def _strides(t: torch.Tensor) -> _Strides:
    assert t.dim() == 4 and t.stride(3) == 1
    return _Strides(t.stride(0), t.stride(1), t.stride(2))


def _mask_struct(mask: MaskSpec) -> _Mask:
    sl = mask.alibi_slopes
    if sl is not None:
        _need_cuda(sl)
        assert sl.dtype == torch.float32 and sl.is_contiguous()
    return _Mask(int(bool(mask.causal)), int(mask.window), sl.data_ptr() if sl is not None else None)


def rope_table(rope_spec: RopeSpec, S: int, device=None) -> Optional[torch.Tensor]:
    """cos/sin table [S + 1, rotary_dim/2, 2] fp32 built on the device (None when rotary_dim == 0);
    the last row is the trailer of step constants."""
    if rope_spec.rotary_dim == 0:
        return None
    n = lib().attnfuse_rope_table_bytes(S, rope_spec.rotary_dim)
    device = device or torch.device("cuda", torch.cuda.current_device())
    table = torch.empty(n // 4, dtype=torch.float32, device=device)
    r = _Rope(rope_spec.theta, rope_spec.rotary_dim, rope_spec.pos_offset)
    _check(lib().attnfuse_rope_table(ctypes.byref(r), S, table.data_ptr(), _stream()))
    # the fp32 rows; the buffer behind this view also carries the bf16 copy the forward kernel streams by TMA
    return table[: (S + 1) * rope_spec.rotary_dim].view(S + 1, rope_spec.rotary_dim // 2, 2)


def rope(x: torch.Tensor, rope_spec: RopeSpec, table: Optional[torch.Tensor], inverse: bool = False,
         out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Separate RoPE pass over x [B,H,S,D] bf16 (contiguous)."""
    _need_cuda(x, table, out)
    assert x.dtype == torch.bfloat16 and x.is_contiguous()
    B, H, S, D = x.shape
    out = torch.empty_like(x) if out is None else out
    assert out.dtype == torch.bfloat16 and out.is_contiguous() and out.shape == x.shape
    sh = _Shape(B, H, H, S, D)
    r = _Rope(rope_spec.theta, rope_spec.rotary_dim, rope_spec.pos_offset)
    _check(lib().attnfuse_rope(ctypes.byref(sh), H, x.data_ptr(), out.data_ptr(), ctypes.byref(r),
                               table.data_ptr() if table is not None else None, int(bool(inverse)), _stream()))
    return out


def fwd(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, rope_spec: RopeSpec, table: Optional[torch.Tensor],
        mask: MaskSpec, softmax_scale: float, out: Optional[torch.Tensor] = None,
        lse: Optional[torch.Tensor] = None, out_dtype: torch.dtype = torch.bfloat16, want_lse: bool = True):
    """Fused forward.  q [B,Hq,S,D], k/v [B,Hkv,S,D] bf16 (last dim contiguous).  Returns (o, lse)."""
    _need_cuda(q, k, v, table, out, lse)
    assert q.dtype == k.dtype == v.dtype == torch.bfloat16
    B, Hq, S, D = q.shape
    Hkv = k.shape[1]
    assert k.shape == v.shape == (B, Hkv, S, D) and k.stride() == v.stride()
    if out is None:
        out = torch.empty((B, Hq, S, D), dtype=out_dtype, device=q.device)
    if lse is None and want_lse:
        lse = torch.empty((B, Hq, S), dtype=torch.float32, device=q.device)
    assert out.is_contiguous() and out.dtype in (torch.bfloat16, torch.float32)
    sh = _Shape(B, Hq, Hkv, S, D)
    sq, skv = _strides(q), _strides(k)
    r = _Rope(rope_spec.theta, rope_spec.rotary_dim, rope_spec.pos_offset)
    m = _mask_struct(mask)
    _check(lib().attnfuse_fwd(ctypes.byref(sh), q.data_ptr(), k.data_ptr(), v.data_ptr(), ctypes.byref(sq),
                              ctypes.byref(skv), ctypes.byref(r), table.data_ptr() if table is not None else None,
                              ctypes.byref(m), Hq // Hkv, float(softmax_scale), out.data_ptr(),
                              AF_F32 if out.dtype == torch.float32 else AF_BF16,
                              lse.data_ptr() if lse is not None else None, _stream()))
    return out, lse


def fwd_variant(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, rope_spec: RopeSpec, table: Optional[torch.Tensor],
                mask: MaskSpec, softmax_scale: float, bias: Optional[torch.Tensor] = None, normaliser: str = "softmax",
                blocks: Optional["BlockMask"] = None, out: Optional[torch.Tensor] = None,
                out_dtype: torch.dtype = torch.bfloat16):
    """Forward of a composed variant (Section 3.1): `fwd` plus an optional additive bias (fp32 [1|B, 1|Hq, S, S]
    on the device), the normaliser ("softmax" or "relu") and optional block lists.  Returns (o, lse); for the ReLU
    normaliser `lse` holds n_i, the number of kept pairs of each row (what `bwd_variant` needs)."""
    _need_cuda(q, k, v, table, out, bias)
    assert q.dtype == k.dtype == v.dtype == torch.bfloat16 and normaliser in ("softmax", "relu")
    B, Hq, S, D = q.shape
    Hkv = k.shape[1]
    assert k.shape == v.shape == (B, Hkv, S, D) and k.stride() == v.stride()
    if out is None:
        out = torch.empty((B, Hq, S, D), dtype=out_dtype, device=q.device)
    relu = normaliser == "relu"
    lse = torch.empty((B, Hq, S), dtype=torch.float32, device=q.device)
    if bias is not None:
        assert bias.dtype == torch.float32 and bias.is_contiguous() and bias.dim() == 4 and bias.shape[2:] == (S, S)
    sh = _Shape(B, Hq, Hkv, S, D)
    sq, skv = _strides(q), _strides(k)
    bl = blocks.struct() if blocks is not None else None
    var = _Variant(_Rope(rope_spec.theta, rope_spec.rotary_dim, rope_spec.pos_offset),
                   table.data_ptr() if table is not None else None, _mask_struct(mask),
                   bias.data_ptr() if bias is not None else None,
                   bias.shape[0] if bias is not None else 1, bias.shape[1] if bias is not None else 1,
                   1 if relu else 0, ctypes.pointer(bl) if bl is not None else None)
    _check(lib().attnfuse_fwd_variant(ctypes.byref(sh), q.data_ptr(), k.data_ptr(), v.data_ptr(), ctypes.byref(sq),
                                      ctypes.byref(skv), ctypes.byref(var), Hq // Hkv, float(softmax_scale),
                                      out.data_ptr(), AF_F32 if out.dtype == torch.float32 else AF_BF16,
                                      lse.data_ptr() if lse is not None else None, _stream()))
    return out, lse


def bwd_variant(q, k, v, o, lse, d_o, rope_spec: RopeSpec, table, mask: MaskSpec, softmax_scale: float,
                bias: Optional[torch.Tensor] = None, normaliser: str = "softmax", blocks: Optional["BlockMask"] = None,
                dq_dtype: torch.dtype = torch.bfloat16, dkv_dtype: torch.dtype = torch.float32, workspace=None):
    """Backward of a composed variant; `lse` is what `fwd_variant` returned for the same variant.
    Returns (dq, dk, dv)."""
    _need_cuda(q, k, v, o, lse, d_o, table, workspace, bias)
    assert normaliser in ("softmax", "relu")
    B, Hq, S, D = q.shape
    Hkv = k.shape[1]
    assert o.is_contiguous() and d_o.is_contiguous() and lse.is_contiguous()
    assert o.dtype == d_o.dtype == torch.bfloat16 and lse.dtype == torch.float32
    if bias is not None:
        assert bias.dtype == torch.float32 and bias.is_contiguous() and bias.dim() == 4 and bias.shape[2:] == (S, S)
    sh = _Shape(B, Hq, Hkv, S, D)
    if workspace is None:
        plain = bias is None and normaliser == "softmax" and blocks is None
        workspace = torch.empty(bwd_workspace_bytes(B, Hq, Hkv, S, D, onepass=plain), dtype=torch.uint8, device=q.device)
    dq = torch.empty((B, Hq, S, D), dtype=dq_dtype, device=q.device)
    dk = torch.empty((B, Hkv, S, D), dtype=dkv_dtype, device=q.device)
    dv = torch.empty((B, Hkv, S, D), dtype=dkv_dtype, device=q.device)
    sq, skv = _strides(q), _strides(k)
    bl = blocks.struct() if blocks is not None else None
    var = _Variant(_Rope(rope_spec.theta, rope_spec.rotary_dim, rope_spec.pos_offset),
                   table.data_ptr() if table is not None else None, _mask_struct(mask),
                   bias.data_ptr() if bias is not None else None,
                   bias.shape[0] if bias is not None else 1, bias.shape[1] if bias is not None else 1,
                   1 if normaliser == "relu" else 0, ctypes.pointer(bl) if bl is not None else None)
    code = lambda dt: AF_F32 if dt == torch.float32 else AF_BF16
    _check(lib().attnfuse_bwd_variant(ctypes.byref(sh), q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                      lse.data_ptr(), d_o.data_ptr(), ctypes.byref(sq), ctypes.byref(skv), ctypes.byref(var),
                                      Hq // Hkv, float(softmax_scale), dq.data_ptr(), code(dq_dtype), dk.data_ptr(),
                                      dv.data_ptr(), code(dkv_dtype), workspace.data_ptr(), workspace.numel(), _stream()))
    return dq, dk, dv


def fwd_fp8(q8: torch.Tensor, k8: torch.Tensor, vt8: torch.Tensor, mask: MaskSpec, softmax_scale: float,
            scale_q: float = 1.0, scale_k: float = 1.0, scale_v: float = 1.0, out_dtype: torch.dtype = torch.bfloat16):
    """Forward with E4M3 operands: q8 [B,Hq,S,D], k8 [B,Hkv,S,D], vt8 [B,Hkv,D,S] (V transposed) as uint8 codes (or
    torch.float8_e4m3fn tensors) on the device, value = code x scale.  Returns (o, lse)."""
    _need_cuda(q8, k8, vt8)
    q8, k8, vt8 = (t.view(torch.uint8) if t.dtype != torch.uint8 else t for t in (q8, k8, vt8))
    assert q8.is_contiguous() and k8.is_contiguous() and vt8.is_contiguous()
    B, Hq, S, D = q8.shape
    Hkv = k8.shape[1]
    assert k8.shape == (B, Hkv, S, D) and vt8.shape == (B, Hkv, D, S)
    out = torch.empty((B, Hq, S, D), dtype=out_dtype, device=q8.device)
    lse = torch.empty((B, Hq, S), dtype=torch.float32, device=q8.device)
    sh = _Shape(B, Hq, Hkv, S, D)
    m = _mask_struct(mask)
    _check(lib().attnfuse_fwd_fp8(ctypes.byref(sh), q8.data_ptr(), k8.data_ptr(), vt8.data_ptr(), ctypes.byref(m), Hq // Hkv,
                                  float(softmax_scale), float(scale_q), float(scale_k), float(scale_v), out.data_ptr(),
                                  AF_F32 if out.dtype == torch.float32 else AF_BF16, lse.data_ptr(), _stream()))
    return out, lse


def fwd_hybrid(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, rope_spec: RopeSpec, table: Optional[torch.Tensor],
               mask: MaskSpec, softmax_scale: float, out: Optional[torch.Tensor] = None,
               lse: Optional[torch.Tensor] = None, out_dtype: torch.dtype = torch.bfloat16, want_lse: bool = True,
               workspace: Optional[torch.Tensor] = None):
    """Hybrid forward (Section 5.3): K rotated once by a RoPE pass into `workspace` (uint8, at least
    attnfuse_fwd_hybrid_workspace_bytes; allocated when None), Q rotated inside the kernel.  Returns (o, lse)."""
    _need_cuda(q, k, v, table, out, lse, workspace)
    assert q.dtype == k.dtype == v.dtype == torch.bfloat16
    B, Hq, S, D = q.shape
    Hkv = k.shape[1]
    assert k.shape == v.shape == (B, Hkv, S, D) and k.stride() == v.stride()
    if out is None:
        out = torch.empty((B, Hq, S, D), dtype=out_dtype, device=q.device)
    if lse is None and want_lse:
        lse = torch.empty((B, Hq, S), dtype=torch.float32, device=q.device)
    assert out.is_contiguous() and out.dtype in (torch.bfloat16, torch.float32)
    sh = _Shape(B, Hq, Hkv, S, D)
    if workspace is None:
        workspace = torch.empty(lib().attnfuse_fwd_hybrid_workspace_bytes(ctypes.byref(sh)), dtype=torch.uint8,
                                device=q.device)
    sq, skv = _strides(q), _strides(k)
    r = _Rope(rope_spec.theta, rope_spec.rotary_dim, rope_spec.pos_offset)
    m = _mask_struct(mask)
    _check(lib().attnfuse_fwd_hybrid(ctypes.byref(sh), q.data_ptr(), k.data_ptr(), v.data_ptr(), ctypes.byref(sq),
                                     ctypes.byref(skv), ctypes.byref(r),
                                     table.data_ptr() if table is not None else None, ctypes.byref(m), Hq // Hkv,
                                     float(softmax_scale), out.data_ptr(),
                                     AF_F32 if out.dtype == torch.float32 else AF_BF16,
                                     lse.data_ptr() if lse is not None else None, workspace.data_ptr(),
                                     workspace.numel() * workspace.element_size(), _stream()))
    return out, lse


class BlockMask:
    """Active 128 x 128 blocks of a block-sparse mask (Section 4.3) as device index lists: CSR by query row
    block and CSC by key block.  Built once from a boolean [nb, nb] matrix (nb = ceil(S / 128))."""

    def __init__(self, active, device="cuda"):
        a = torch.as_tensor(active).to(torch.bool).cpu()
        assert a.dim() == 2 and a.shape[0] == a.shape[1]
        self.nb = a.shape[0]
        self.active = a
        counts = a.sum(1).to(torch.int32)
        self.row_ptr = torch.cat([torch.zeros(1, dtype=torch.int32), counts.cumsum(0).to(torch.int32)]).to(device)
        self.col_idx = a.nonzero()[:, 1].to(torch.int32).contiguous().to(device)
        at = a.t().contiguous()
        counts_t = at.sum(1).to(torch.int32)
        self.col_ptr = torch.cat([torch.zeros(1, dtype=torch.int32), counts_t.cumsum(0).to(torch.int32)]).to(device)
        self.row_idx = at.nonzero()[:, 1].to(torch.int32).contiguous().to(device)
        # launch orders: longest lists first
        self.row_order = torch.argsort(counts, descending=True, stable=True).to(torch.int32).to(device)
        self.col_order = torch.argsort(counts_t, descending=True, stable=True).to(torch.int32).to(device)
        # lists by pair of row blocks (2r, 2r + 1): sorted union, bit 28 / 29 = listed by the first / second row block
        an = a.numpy()
        ptr, idx = [0], []
        for r in range(0, self.nb, 2):
            first = an[r]
            second = an[r + 1] if r + 1 < self.nb else first & False
            for j in (first | second).nonzero()[0]:
                idx.append(int(j) | (int(first[j]) << 28) | (int(second[j]) << 29))
            ptr.append(len(idx))
        self.pair_ptr = torch.tensor(ptr, dtype=torch.int32).to(device)
        self.pair_idx = torch.tensor(idx if idx else [0], dtype=torch.int32).to(device)
        plen = torch.tensor(ptr[1:], dtype=torch.int64) - torch.tensor(ptr[:-1], dtype=torch.int64)
        self.pair_order = torch.argsort(plen, descending=True, stable=True).to(torch.int32).to(device)
        if self.col_idx.numel() == 0:   # keep the pointers valid
            self.col_idx = torch.zeros(1, dtype=torch.int32, device=device)
            self.row_idx = torch.zeros(1, dtype=torch.int32, device=device)

    def struct(self):
        return _Blocks(128, self.row_ptr.data_ptr(), self.col_idx.data_ptr(), self.col_ptr.data_ptr(),
                       self.row_idx.data_ptr(), self.row_order.data_ptr(), self.col_order.data_ptr(),
                       self.pair_ptr.data_ptr(), self.pair_idx.data_ptr(), self.pair_order.data_ptr())


def fwd_blocks(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, rope_spec: RopeSpec, table: Optional[torch.Tensor],
               mask: MaskSpec, softmax_scale: float, blocks: BlockMask, out: Optional[torch.Tensor] = None,
               lse: Optional[torch.Tensor] = None, out_dtype: torch.dtype = torch.bfloat16):
    """Block-sparse forward: `fwd` restricted to the active blocks of `blocks`.  Returns (o, lse)."""
    _need_cuda(q, k, v, table, out, lse)
    assert q.dtype == k.dtype == v.dtype == torch.bfloat16
    B, Hq, S, D = q.shape
    Hkv = k.shape[1]
    assert k.shape == v.shape == (B, Hkv, S, D) and k.stride() == v.stride()
    assert blocks.nb == (S + 127) // 128
    if out is None:
        out = torch.empty((B, Hq, S, D), dtype=out_dtype, device=q.device)
    if lse is None:
        lse = torch.empty((B, Hq, S), dtype=torch.float32, device=q.device)
    sh = _Shape(B, Hq, Hkv, S, D)
    sq, skv = _strides(q), _strides(k)
    r = _Rope(rope_spec.theta, rope_spec.rotary_dim, rope_spec.pos_offset)
    m = _mask_struct(mask)
    bl = blocks.struct()
    _check(lib().attnfuse_fwd_blocks(ctypes.byref(sh), q.data_ptr(), k.data_ptr(), v.data_ptr(), ctypes.byref(sq),
                                     ctypes.byref(skv), ctypes.byref(r), table.data_ptr() if table is not None else None,
                                     ctypes.byref(m), Hq // Hkv, float(softmax_scale), ctypes.byref(bl), out.data_ptr(),
                                     AF_F32 if out.dtype == torch.float32 else AF_BF16, lse.data_ptr(), _stream()))
    return out, lse


def fwd_host(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, rope_spec: RopeSpec, table: Optional[torch.Tensor],
             mask: MaskSpec, softmax_scale: float, out: torch.Tensor, lse: Optional[torch.Tensor],
             staging: torch.Tensor):
    """Forward with HOST (pinned) q, k, v, out, lse; `staging` is a device byte buffer."""
    for t in (q, k, v, out):
        assert not t.is_cuda and t.is_contiguous() and t.dtype == torch.bfloat16
    _need_cuda(staging, table)
    B, Hq, S, D = q.shape
    Hkv = k.shape[1]
    sh = _Shape(B, Hq, Hkv, S, D)
    r = _Rope(rope_spec.theta, rope_spec.rotary_dim, rope_spec.pos_offset)
    m = _mask_struct(mask)
    _check(lib().attnfuse_fwd_host(ctypes.byref(sh), q.data_ptr(), k.data_ptr(), v.data_ptr(), ctypes.byref(r),
                                   table.data_ptr() if table is not None else None, ctypes.byref(m), Hq // Hkv,
                                   float(softmax_scale), out.data_ptr(),
                                   lse.data_ptr() if lse is not None else None, staging.data_ptr(),
                                   staging.numel() * staging.element_size(), _stream()))
    return out, lse


def fwd_host_staging_bytes(B: int, Hq: int, Hkv: int, S: int, D: int) -> int:
    sh = _Shape(B, Hq, Hkv, S, D)
    return lib().attnfuse_fwd_host_staging_bytes(ctypes.byref(sh))


def bwd_workspace_bytes(B: int, Hq: int, Hkv: int, S: int, D: int, onepass: bool = True) -> int:
    """Workspace size of the backward: with `onepass` the size that admits the one-pass sequence (delta, both
    rotated caches and the fp32 dQ accumulator), otherwise delta and the two caches."""
    sh = _Shape(B, Hq, Hkv, S, D)
    if onepass:
        return lib().attnfuse_bwd_onepass_workspace_bytes(ctypes.byref(sh))
    return lib().attnfuse_bwd_workspace_bytes(ctypes.byref(sh))


def bwd(q, k, v, o, lse, d_o, rope_spec: RopeSpec, table, mask: MaskSpec, softmax_scale: float,
        dq_dtype: torch.dtype = torch.bfloat16, dkv_dtype: torch.dtype = torch.float32, workspace=None,
        blocks: Optional[BlockMask] = None):
    """Fused backward (over the active blocks of `blocks`, if given).  Returns (dq, dk, dv).
    Without a workspace of the caller's, one of the largest useful size is allocated (`bwd_workspace_bytes`)."""
    _need_cuda(q, k, v, o, lse, d_o, table, workspace)
    B, Hq, S, D = q.shape
    Hkv = k.shape[1]
    assert o.is_contiguous() and d_o.is_contiguous() and lse.is_contiguous()
    assert o.dtype == d_o.dtype == torch.bfloat16 and lse.dtype == torch.float32
    sh = _Shape(B, Hq, Hkv, S, D)
    if workspace is None:
        workspace = torch.empty(bwd_workspace_bytes(B, Hq, Hkv, S, D), dtype=torch.uint8, device=q.device)
    dq = torch.empty((B, Hq, S, D), dtype=dq_dtype, device=q.device)
    dk = torch.empty((B, Hkv, S, D), dtype=dkv_dtype, device=q.device)
    dv = torch.empty((B, Hkv, S, D), dtype=dkv_dtype, device=q.device)
    sq, skv = _strides(q), _strides(k)
    r = _Rope(rope_spec.theta, rope_spec.rotary_dim, rope_spec.pos_offset)
    m = _mask_struct(mask)
    code = lambda dt: AF_F32 if dt == torch.float32 else AF_BF16
    if blocks is not None:
        assert blocks.nb == (S + 127) // 128
        bl = blocks.struct()
        _check(lib().attnfuse_bwd_blocks(ctypes.byref(sh), q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                         lse.data_ptr(), d_o.data_ptr(), ctypes.byref(sq), ctypes.byref(skv),
                                         ctypes.byref(r), table.data_ptr() if table is not None else None,
                                         ctypes.byref(m), Hq // Hkv, float(softmax_scale), ctypes.byref(bl),
                                         dq.data_ptr(), code(dq_dtype), dk.data_ptr(), dv.data_ptr(), code(dkv_dtype),
                                         workspace.data_ptr(), workspace.numel(), _stream()))
        return dq, dk, dv
    _check(lib().attnfuse_bwd(ctypes.byref(sh), q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                              lse.data_ptr(), d_o.data_ptr(), ctypes.byref(sq), ctypes.byref(skv), ctypes.byref(r),
                              table.data_ptr() if table is not None else None, ctypes.byref(m), Hq // Hkv,
                              float(softmax_scale), dq.data_ptr(), code(dq_dtype), dk.data_ptr(), dv.data_ptr(),
                              code(dkv_dtype), workspace.data_ptr(), workspace.numel(), _stream()))
    return dq, dk, dv


BWD_STATIC_MAX_ROWS = 1 << 20


def decode(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, mask: MaskSpec, softmax_scale: float,
           n_splits: int = 0, out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
           workspace: Optional[torch.Tensor] = None, want_lse: bool = True):
    """Flash Decoding: q [B,Hq,D] (one position per head, the last one) against the cache k/v [B,Hkv,N,D].
    Returns (o [B,Hq,D] bf16, lse [B,Hq])."""
    _need_cuda(q, k, v, out, lse, workspace)
    assert q.dtype == k.dtype == v.dtype == torch.bfloat16 and q.is_contiguous()
    B, Hq, D = q.shape
    Hkv, N = k.shape[1], k.shape[2]
    assert k.shape == v.shape == (B, Hkv, N, D) and k.stride() == v.stride()
    if out is None:
        out = torch.empty((B, Hq, D), dtype=torch.bfloat16, device=q.device)
    if lse is None and want_lse:
        lse = torch.empty((B, Hq), dtype=torch.float32, device=q.device)
    sh = _Shape(B, Hq, Hkv, N, D)
    if n_splits <= 0:
        n_splits = lib().attnfuse_decode_splits(ctypes.byref(sh))
    if workspace is None:   # (a caller's own workspace must have been cleared once: decode_workspace)
        workspace = torch.zeros(lib().attnfuse_decode_workspace_bytes(ctypes.byref(sh), n_splits), dtype=torch.uint8,
                                device=q.device)
    skv = _strides(k)
    m = _mask_struct(mask)
    _check(lib().attnfuse_decode(ctypes.byref(sh), q.data_ptr(), k.data_ptr(), v.data_ptr(), ctypes.byref(skv),
                                 ctypes.byref(m), Hq // Hkv, float(softmax_scale), out.data_ptr(),
                                 lse.data_ptr() if lse is not None else None, int(n_splits), workspace.data_ptr(),
                                 workspace.numel() * workspace.element_size(), _stream()))
    return out, lse


def decode_workspace(B: int, Hq: int, Hkv: int, N: int, D: int, n_splits: int = 0, device="cuda") -> torch.Tensor:
    """A cleared workspace for `decode` on this geometry (its ticket counters must start at zero)."""
    sh = _Shape(B, Hq, Hkv, N, D)
    ws = torch.empty(lib().attnfuse_decode_workspace_bytes(ctypes.byref(sh), n_splits), dtype=torch.uint8, device=device)
    _check(lib().attnfuse_decode_workspace_init(ws.data_ptr(), ws.numel(), _stream()))
    return ws


def bwd_static(q, k, v, o, lse, d_o, rope_spec: RopeSpec, table, mask: MaskSpec, softmax_scale: float,
               dq: torch.Tensor, dk: torch.Tensor, dv: torch.Tensor):
    """Backward for callers that must not allocate: no workspace argument, the scratch lives inside
    the library (B*Hq*S <= BWD_STATIC_MAX_ROWS).  The caller passes the output tensors; this wrapper
    creates no tensor either.  Calls on one device share that scratch, so do not let two of them
    overlap on the GPU."""
    _need_cuda(q, k, v, o, lse, d_o, table, dq, dk, dv)
    B, Hq, S, D = q.shape
    Hkv = k.shape[1]
    assert o.is_contiguous() and d_o.is_contiguous() and lse.is_contiguous()
    assert dq.is_contiguous() and dk.is_contiguous() and dv.is_contiguous() and dk.dtype == dv.dtype
    assert dq.shape == q.shape and dk.shape == k.shape and dv.shape == v.shape
    sh = _Shape(B, Hq, Hkv, S, D)
    sq, skv = _strides(q), _strides(k)
    r = _Rope(rope_spec.theta, rope_spec.rotary_dim, rope_spec.pos_offset)
    m = _mask_struct(mask)
    code = lambda dt: AF_F32 if dt == torch.float32 else AF_BF16
    _check(lib().attnfuse_bwd_static(ctypes.byref(sh), q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                     lse.data_ptr(), d_o.data_ptr(), ctypes.byref(sq), ctypes.byref(skv),
                                     ctypes.byref(r), table.data_ptr() if table is not None else None,
                                     ctypes.byref(m), Hq // Hkv, float(softmax_scale), dq.data_ptr(), code(dq.dtype),
                                     dk.data_ptr(), dv.data_ptr(), code(dk.dtype), _stream()))
    return dq, dk, dv
