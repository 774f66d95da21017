"""GPU parity of the fp8 forward (E4M3 operands, opt-in): the fp64 oracle is evaluated on the DEQUANTISED inputs, so the
bound below measures the path's own arithmetic (fp8 products are exact in fp32; what rounds is P, to E4M3), not the
input quantisation."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_13612_b200 as af
from paper_2609_13612_b200 import synth

pytestmark = pytest.mark.gpu
W = synth.Workload

# A probability rounded to E4M3 carries up to 2^-4 relative error (three mantissa bits), uniformly spread, so about
# 2^-4 / sqrt(3) = 0.036 rms.  On a row with n comparable weights the errors average and O_i moves by about
# 0.036 |v| / sqrt(n); the worst rows are those with two or three comparable keys, where one weight's rounding reaches
# O at up to (1/2) 2^-4 |v_a - v_b| (|v| up to ~4.5 on unit-variance data: 0.1 at the extreme); a one-key row has none
# (P = 1 exactly).  Measured on these cases and on the Llama-3-8B shape: max 0.05, mean 0.001-0.006.
FP8_MAX_TOL = 1e-1
FP8_MEAN_TOL = 8e-3


def quantise(x):
    """Per-tensor scale so that the largest magnitude lands on 448, codes and dequantised values."""
    scale = float(np.abs(x).max()) / 448.0
    codes = synth.e4m3_encode(x / np.float32(scale))
    return codes, scale, synth.e4m3_decode(codes).astype(np.float64) * scale


CASES = [
    W("fp8_causal_gqa", 2, 8, 2, 512, 128, rotary_dim=0, seed_id=901),
    W("fp8_causal_two_row_blocks", 1, 3, 3, 640, 128, rotary_dim=0, seed_id=902),
    W("fp8_full_ragged", 1, 4, 2, 400, 128, rotary_dim=0, causal=False, seed_id=903),
    W("fp8_window", 1, 4, 1, 768, 128, rotary_dim=0, window=200, seed_id=904),
    W("fp8_short", 1, 2, 2, 16, 128, rotary_dim=0, seed_id=905),
]


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_fp8_forward(w):
    t = synth.draw_all(w)
    q8, sq, dq = quantise(t["q"])
    k8, sk, dk = quantise(t["k"])
    v8, sv, dv = quantise(t["v"])
    vt8 = np.ascontiguousarray(v8.transpose(0, 1, 3, 2))
    mask = af.MaskSpec(causal=w.causal, window=w.window)
    o, lse = af.fwd_fp8(torch.from_numpy(q8).cuda(), torch.from_numpy(k8).cuda(), torch.from_numpy(vt8).cuda(), mask, w.scale,
                        sq, sk, sv, out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    want_o, want_l = oracle.fwd(dq, dk, dv, rotary_dim=0, causal=w.causal, window=w.window, scale=w.scale)
    d = np.abs(o.cpu().numpy().astype(np.float64) - want_o)
    assert np.isfinite(d).all()
    assert d.max() <= FP8_MAX_TOL and d.mean() <= FP8_MEAN_TOL, "%s: max %.4g mean %.4g" % (w.name, d.max(), d.mean())
    # L sums the unrounded probabilities of exact fp8 products: the bf16 path's bound holds with room to spare
    assert np.abs(lse.cpu().numpy() - want_l).max() <= 2e-3
    # row 0 under a causal mask sees one key: P = 1 exactly, O = v_0 up to the output rounding
    if w.causal:
        assert np.abs(o[:, :, 0].cpu().numpy() - want_o[:, :, 0]).max() <= 1e-5


def test_fp8_argument_errors():
    q = torch.zeros((1, 2, 128, 64), dtype=torch.uint8, device="cuda")
    with pytest.raises(af.AttnFuseError) as e:      # D = 64 is not built
        af.fwd_fp8(q, q, q.transpose(2, 3).contiguous(), af.MaskSpec(), 0.125)
    assert e.value.code == 2
    q = torch.zeros((1, 2, 120, 128), dtype=torch.uint8, device="cuda")
    with pytest.raises(af.AttnFuseError) as e:      # S must be a multiple of 16
        af.fwd_fp8(q, q, q.transpose(2, 3).contiguous(), af.MaskSpec(), 0.125)
    assert e.value.code == 2
