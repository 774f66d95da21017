"""The 8-bit E4M3 input conversion of the fp8 entry point (paper_2609_13612_b200.synth): pinned against the format's
definition - hand values - and against torch's own float8_e4m3fn conversion."""
import numpy as np
import torch

from paper_2609_13612_b200 import synth


def test_decode_of_all_codes_matches_torch():
    codes = np.arange(256, dtype=np.uint8)
    mine = synth.e4m3_decode(codes)
    ref = torch.from_numpy(codes).view(torch.float8_e4m3fn).float().numpy()
    assert np.array_equal(np.isnan(mine), np.isnan(ref)) and np.isnan(mine).sum() == 2
    ok = ~np.isnan(ref)
    assert np.array_equal(mine[ok], ref[ok])


def test_hand_values():
    # 1.0 = 0.0111.000; largest finite 448 = 0.1111.110; smallest subnormal 2^-9 = 0.0000.001; smallest normal 2^-6
    assert synth.e4m3_encode(np.array([1.0, 448.0, 2.0 ** -9, 2.0 ** -6, -1.5], np.float32)).tolist() == [0x38, 0x7E, 0x01, 0x08, 0xBC]
    # ties go to the even mantissa: 1.0625 lies between 1.0 and 1.125 -> 1.0; 1.1875 between 1.125 and 1.25 -> 1.25
    assert synth.e4m3_decode(synth.e4m3_encode(np.array([1.0625, 1.1875], np.float32))).tolist() == [1.0, 1.25]
    # saturation instead of NaN, half the smallest subnormal rounds to zero, a mantissa carry moves to the next exponent
    assert synth.e4m3_decode(synth.e4m3_encode(np.array([1e6, -1e6, 2.0 ** -10, 1.97], np.float32))).tolist() == [448.0, -448.0, 0.0, 2.0]


def test_encode_matches_torch_inside_the_finite_range():
    rng = np.random.Generator(np.random.PCG64(7))
    x = np.concatenate([rng.standard_normal(100000).astype(np.float32) * s for s in (1e-3, 0.02, 1.0, 30.0, 150.0)])
    x = x[np.abs(x) <= 448.0]
    mine = synth.e4m3_encode(x)
    ref = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(mine, ref)
    # and the conversion is idempotent on representable values
    assert np.array_equal(synth.e4m3_encode(synth.e4m3_decode(mine)), mine)
