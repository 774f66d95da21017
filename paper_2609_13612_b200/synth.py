"""Seeded synthetic inputs for the fused RoPE + masked attention path.

This module only draws random tensors and describes workloads.  It holds none
of the method's arithmetic (no rotation, no softmax, no masking): both the CUDA
path and the CPU oracle are fed from here so that they see the very same
numbers, and neither implementation can leak into the other through it.

The paper's workloads are random tensors in model geometries (GPT-2-small and
Llama-3-8B attention shapes, Section 6), so seeded N(0, sigma) tensors of those
shapes are the workload itself, not a stand-in for a dataset.

Values are drawn in fp32 and rounded once (round-to-nearest-even) to bf16; the
rounded values are what both sides consume, so input quantisation is never
charged to either side as error.  For the fp8 entry point the same holds one step
further: the inputs are rounded to 8-bit E4M3 codes here (a number-format
conversion, no arithmetic of the method), the CUDA path takes the codes and the
oracle their decoded values.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import numpy as np

BASE_SEED = 20260913
TENSOR_IDS = {"q": 0, "k": 1, "v": 2, "do": 3}


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); result stays fp32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of fp32 values that are already bf16-representable."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16).reshape(x.shape)


def bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """fp32 values of bf16 bit patterns."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16
    return b.view(np.float32).reshape(bits.shape)


def e4m3_decode(codes: np.ndarray) -> np.ndarray:
    """fp32 values of 8-bit E4M3 codes (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no infinities, the one
    NaN pattern S.1111.111; largest finite value 448): the operand format of the fp8 entry point."""
    c = np.ascontiguousarray(codes, dtype=np.uint8).astype(np.int32)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = c & 0x7
    val = np.where(e == 0, m * 2.0 ** -9, (8 + m) * np.exp2(e.astype(np.float64) - 10.0))
    val = np.where((e == 15) & (m == 7), np.nan, val)
    return (sign * val).astype(np.float32).reshape(codes.shape)


def e4m3_encode(x: np.ndarray) -> np.ndarray:
    """8-bit E4M3 codes of fp32 values: round to nearest, ties to even, saturating at +-448."""
    x = np.ascontiguousarray(x, dtype=np.float32).astype(np.float64)
    sign = np.signbit(x)
    a = np.minimum(np.abs(x), 448.0)
    # exponent of the spacing: values below 2^-6 share the subnormal spacing 2^-9
    e = np.floor(np.log2(np.maximum(a, 2.0 ** -6)))
    e = np.clip(e, -6, 8)
    step = np.exp2(e - 3)
    q = np.rint(a / step)                      # numpy rounds halves to even
    # a mantissa that rounded up to 16 steps moves to the next exponent
    bump = q >= 16
    e = np.where(bump, e + 1, e)
    q = np.where(bump, 8, q)
    sub = a < 2.0 ** -6
    qs = np.rint(a / 2.0 ** -9)                # subnormal range: 0 .. 8 steps of 2^-9 (8 is the smallest normal)
    code = np.where(sub, np.where(qs >= 8, 0x08, qs), ((e + 7).astype(np.int64) << 3) | (q.astype(np.int64) - 8))
    code = np.minimum(code.astype(np.int64), 0x7E)
    return (code | (sign.astype(np.int64) << 7)).astype(np.uint8).reshape(x.shape)


@dataclasses.dataclass(frozen=True)
class Workload:
    """One attention problem: geometry plus the composed variant's parameters."""

    name: str
    B: int
    Hq: int
    Hkv: int
    S: int
    D: int
    theta: float = 10000.0
    rotary_dim: int = -1  # -1: all D dims; 0: no RoPE
    pos_offset: int = 0
    causal: bool = True
    window: int = -1  # < 0: none
    alibi: bool = False
    sigma: float = 1.0
    seed_id: int = 0
    backward: bool = False

    @property
    def R(self) -> int:
        return self.D if self.rotary_dim < 0 else self.rotary_dim

    @property
    def group(self) -> int:
        return self.Hq // self.Hkv

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.D)

    def kept_pairs_per_head(self) -> int:
        """Number of (query, key) pairs the mask keeps, per head."""
        S, W = self.S, self.window
        if self.causal:
            if W < 0 or W >= S - 1:
                return S * (S + 1) // 2
            return (W + 1) * (W + 2) // 2 + (S - W - 1) * (W + 1)
        if W < 0 or W >= S - 1:
            return S * S
        return S * (2 * W + 1) - W * (W + 1)

    def fwd_flops(self) -> float:
        """Algorithmic forward FLOPs: two contractions over the kept pairs only."""
        return 4.0 * self.D * self.kept_pairs_per_head() * self.B * self.Hq

    def bwd_flops(self) -> float:
        """Algorithmic backward FLOPs: five contractions over the kept pairs."""
        return 2.5 * self.fwd_flops()

    def alibi_slopes(self) -> Optional[np.ndarray]:
        """Geometric slopes 2^(-8h/Hq), h = 1..Hq (fp32), or None."""
        if not self.alibi:
            return None
        h = np.arange(1, self.Hq + 1, dtype=np.float64)
        return np.exp2(-8.0 * h / self.Hq).astype(np.float32)


# The five benchmark configurations, in order.  CONFIGS[1] is the one the
# headline metric is quoted on.
CONFIGS = (
    Workload("c1_tiny_rope_causal", B=1, Hq=2, Hkv=2, S=128, D=64, theta=1.0e4, seed_id=1),
    Workload("c2_llama3_8b_fwd", B=1, Hq=32, Hkv=8, S=4096, D=128, theta=5.0e5, seed_id=2),
    Workload("c3_composed_window_alibi", B=2, Hq=16, Hkv=16, S=8192, D=128, theta=1.0e4,
             window=1024, alibi=True, seed_id=3),
    Workload("c4_long_context", B=1, Hq=32, Hkv=8, S=32768, D=128, theta=5.0e5, sigma=0.5, seed_id=4),
    Workload("c5_llama3_8b_train", B=4, Hq=32, Hkv=8, S=2048, D=128, theta=5.0e5, seed_id=5,
             backward=True),
)


def draw(w: Workload, which: str) -> np.ndarray:
    """Tensor `which` in {"q","k","v","do"} of workload `w`: fp32 array holding
    bf16-representable values, layout [B, H, S, D] contiguous."""
    tid = TENSOR_IDS[which]
    H = w.Hq if which in ("q", "do") else w.Hkv
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([BASE_SEED, w.seed_id, tid])))
    x = rng.standard_normal((w.B, H, w.S, w.D), dtype=np.float32)
    if w.sigma != 1.0:
        x *= np.float32(w.sigma)
    return round_to_bf16(x)


def draw_all(w: Workload) -> dict:
    out = {n: draw(w, n) for n in ("q", "k", "v")}
    if w.backward:
        out["do"] = draw(w, "do")
    return out
