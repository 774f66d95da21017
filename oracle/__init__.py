"""fp64 CPU oracle of the fused RoPE + masked attention path (ctypes binding).

TEST INFRASTRUCTURE ONLY.  Nothing on the product path imports this package; only
tests, the smoke check and the bench's cpu_baseline / reference arm do.  It shares no
code with the CUDA library.  The arithmetic lives in attn_oracle.c (the plain
definition in fp64); this file only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

from .build import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int)
        i, d = ctypes.c_int, ctypes.c_double
        lib.af_oracle_rope.argtypes = [dp, dp, i, i, i, i, d, i, i, i]
        lib.af_oracle_rope.restype = None
        lib.af_oracle_fwd.argtypes = [dp, dp, dp, i, i, i, i, i, d, i, i, i, i, dp, d, ip, i, dp, dp]
        lib.af_oracle_fwd.restype = None
        lib.af_oracle_bwd.argtypes = [dp, dp, dp, dp, i, i, i, i, i, d, i, i, i, i, dp, d, dp, dp, dp]
        lib.af_oracle_bwd.restype = None
        bp = ctypes.POINTER(ctypes.c_ubyte)
        lib.af_oracle_fwd_blocks.argtypes = [dp, dp, dp, i, i, i, i, i, d, i, i, i, i, dp, d, bp, i, ip, i, dp, dp]
        lib.af_oracle_fwd_blocks.restype = None
        lib.af_oracle_bwd_blocks.argtypes = [dp, dp, dp, dp, i, i, i, i, i, d, i, i, i, i, dp, d, bp, i, dp, dp, dp]
        lib.af_oracle_bwd_blocks.restype = None
        lib.af_oracle_fwd_variant.argtypes = [dp, dp, dp, i, i, i, i, i, d, i, i, i, i, dp, d, bp, i, dp, i, i, i, ip, i, dp, dp]
        lib.af_oracle_fwd_variant.restype = None
        lib.af_oracle_bwd_variant.argtypes = [dp, dp, dp, dp, i, i, i, i, i, d, i, i, i, i, dp, d, bp, i, dp, i, i, i, dp, dp, dp]
        lib.af_oracle_bwd_variant.restype = None
        _lib = lib
    return _lib


def _f64(x) -> np.ndarray:
    return np.ascontiguousarray(x, dtype=np.float64)


def _p(a: Optional[np.ndarray]):
    if a is None:
        return None
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def rope(x, theta: float, rotary_dim: int, pos_offset: int = 0, inverse: bool = False) -> np.ndarray:
    """Rotate every row of x [B,H,S,D] (Section 4.1; NeoX half-swap pairing)."""
    x = _f64(x)
    B, H, S, D = x.shape
    assert rotary_dim % 2 == 0 and 0 <= rotary_dim <= D
    y = np.empty_like(x)
    _load().af_oracle_rope(_p(x), _p(y), B, H, S, D, float(theta), int(rotary_dim), int(pos_offset),
                           int(bool(inverse)))
    return y


def _check(q, k, v):
    B, Hq, S, D = q.shape
    Bk, Hkv, Sk, Dk = k.shape
    assert (Bk, Sk, Dk) == (B, S, D) and v.shape == k.shape and Hq % Hkv == 0
    return B, Hq, Hkv, S, D


def _blocks(blocks, block_size, S):
    """Active-block matrix [nb, nb] (Section 4.3) as contiguous bytes, or None."""
    if blocks is None:
        return None, None
    nb = (S + block_size - 1) // block_size
    a = np.ascontiguousarray(np.asarray(blocks) != 0, dtype=np.uint8)
    assert a.shape == (nb, nb) and block_size > 0
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_ubyte))


def _bias(bias, B, Hq, S):
    """additive_bias (Section 3.1): [Bb, Hb, S, S] with Bb in {1, B}, Hb in {1, Hq}, or None."""
    if bias is None:
        return None, 1, 1
    a = _f64(bias)
    assert a.ndim == 4 and a.shape[2:] == (S, S) and a.shape[0] in (1, B) and a.shape[1] in (1, Hq)
    return a, a.shape[0], a.shape[1]


def fwd(q, k, v, *, theta: float = 10000.0, rotary_dim: int = 0, pos_offset: int = 0,
        causal: bool = True, window: int = -1, slopes=None, scale: Optional[float] = None,
        rows: Optional[Sequence[int]] = None, blocks=None, block_size: int = 128, bias=None,
        normaliser: str = "softmax"):
    """O and L = m + ln(l) of the composed variant.  `rows`: optional subset of query
    rows (same for every head); then O is [B,Hq,len(rows),D].  `blocks`: optional [nb, nb] matrix of
    active blocks (Section 4.3): pairs in inactive blocks are dropped on top of the element mask.
    `bias`: additive_bias of Section 3.1.  normaliser "relu": relu_attention of Section 3.1 (L is None)."""
    assert normaliser in ("softmax", "relu")
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, Hq, Hkv, S, D = _check(q, k, v)
    scale = float(scale) if scale is not None else 1.0 / np.sqrt(D)
    sl = None if slopes is None else _f64(slopes)
    if sl is not None:
        assert sl.shape == (Hq,)
    if rows is None:
        nr, rp = S, None
    else:
        ra = np.ascontiguousarray(rows, dtype=np.int32)
        assert ra.ndim == 1 and (ra >= 0).all() and (ra < S).all()
        nr, rp = len(ra), ra.ctypes.data_as(ctypes.POINTER(ctypes.c_int))
    o = np.empty((B, Hq, nr, D), dtype=np.float64)
    lse = np.empty((B, Hq, nr), dtype=np.float64)
    ba, bptr = _blocks(blocks, block_size, S)
    bi, bi_b, bi_h = _bias(bias, B, Hq, S)
    relu = normaliser == "relu"
    _load().af_oracle_fwd_variant(_p(q), _p(k), _p(v), B, Hq, Hkv, S, D, float(theta), int(rotary_dim),
                                  int(pos_offset), int(bool(causal)), int(window), _p(sl), scale,
                                  bptr, int(block_size), _p(bi), bi_b, bi_h, int(relu), rp, nr, _p(o), _p(lse))
    return o, (None if relu else lse)


def bwd(q, k, v, d_o, *, theta: float = 10000.0, rotary_dim: int = 0, pos_offset: int = 0,
        causal: bool = True, window: int = -1, slopes=None, scale: Optional[float] = None,
        blocks=None, block_size: int = 128, bias=None, normaliser: str = "softmax"):
    """dQ, dK, dV for upstream dO (Section 4.4 algebra, rotation transposed back).  The bias gets no gradient."""
    assert normaliser in ("softmax", "relu")
    q, k, v, d_o = _f64(q), _f64(k), _f64(v), _f64(d_o)
    B, Hq, Hkv, S, D = _check(q, k, v)
    assert d_o.shape == q.shape
    scale = float(scale) if scale is not None else 1.0 / np.sqrt(D)
    sl = None if slopes is None else _f64(slopes)
    dq = np.empty_like(q)
    dk = np.empty_like(k)
    dv = np.empty_like(v)
    ba, bptr = _blocks(blocks, block_size, S)
    bi, bi_b, bi_h = _bias(bias, B, Hq, S)
    _load().af_oracle_bwd_variant(_p(q), _p(k), _p(v), _p(d_o), B, Hq, Hkv, S, D, float(theta), int(rotary_dim),
                                  int(pos_offset), int(bool(causal)), int(window), _p(sl), scale,
                                  bptr, int(block_size), _p(bi), bi_b, bi_h, int(normaliser == "relu"),
                                  _p(dq), _p(dk), _p(dv))
    return dq, dk, dv


def run_workload(w, tensors, rows=None, backward=False):
    """Run a synth.Workload description through the oracle."""
    kw = dict(theta=w.theta, rotary_dim=w.R, pos_offset=w.pos_offset, causal=w.causal,
              window=w.window, slopes=w.alibi_slopes(), scale=w.scale)
    if backward:
        return bwd(tensors["q"], tensors["k"], tensors["v"], tensors["do"], **kw)
    return fwd(tensors["q"], tensors["k"], tensors["v"], rows=rows, **kw)
