"""GPU parity of the composed-variant entry point (Section 3.1): additive_bias, relu_attention and `full`, alone and
composed with rope / causal / sliding_window / alibi / block_sparse, against the fp64 oracle on the same inputs."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_13612_b200 as af
from paper_2609_13612_b200 import synth
import parity_util as pu

pytestmark = pytest.mark.gpu
W = synth.Workload


def bias_of(w, shape_b, shape_h, seed, minus_inf_fraction=0.0):
    """Seeded fp32 bias [shape_b, shape_h, S, S], N(0, 0.5), optionally with some entries at -inf."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([synth.BASE_SEED, w.seed_id, 7, seed])))
    b = (0.5 * rng.standard_normal((shape_b, shape_h, w.S, w.S))).astype(np.float32)
    if minus_inf_fraction > 0:
        drop = rng.random(b.shape) < minus_inf_fraction
        drop[..., np.arange(w.S), np.arange(w.S)] = False      # keep the diagonal: no empty rows
        b[drop] = -np.inf
    return b


def run(w, bias=None, normaliser="softmax", out_dtype=torch.bfloat16):
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S) if w.R > 0 else None
    o, lse = af.fwd_variant(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale,
                            bias=torch.from_numpy(bias).cuda() if bias is not None else None, normaliser=normaliser,
                            out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    want_o, want_l = oracle.fwd(t["q"], t["k"], t["v"], theta=w.theta, rotary_dim=w.R, pos_offset=w.pos_offset,
                                causal=w.causal, window=w.window, slopes=w.alibi_slopes(), scale=w.scale, bias=bias,
                                normaliser=normaliser)
    if normaliser == "relu":
        # The ReLU normaliser passes the score itself to the output: O_i = sum_j max(s_ij, 0) v_j / n_i.  The error of
        # a score (bf16 roundings of q' and k': up to about 1e-2 over this many rows, see LSE_TOL) and the bf16
        # rounding of the unnormalised weight (2^-9 of values up to ~5) reach O multiplied by |v| (up to ~4.5 here)
        # and undivided where a row keeps a single pair; the softmax maps such a row to P = 1 exactly.  Hence a
        # stated bound of its own for this combinator: 6e-2 max, the common 2e-3 mean.
        pu.assert_close("%s O (%s)" % (w.name, normaliser), pu.to_np(o), want_o, max_tol=6e-2)
    else:
        pu.assert_close("%s O (%s)" % (w.name, normaliser), pu.to_np(o), want_o)
    if normaliser == "softmax":
        assert np.abs(pu.to_np(lse) - want_l).max() <= pu.LSE_TOL
    else:
        assert lse is None and want_l is None
    return o


BIAS_CASES = [
    (W("bias_causal_gqa", 2, 4, 2, 384, 128, theta=5e5, seed_id=701), "full", 0.0),
    (W("bias_broadcast_heads", 2, 4, 2, 300, 128, theta=1e4, seed_id=702), "per_batch", 0.0),
    (W("bias_broadcast_all_d64", 1, 6, 2, 515, 64, theta=1e4, seed_id=703), "shared", 0.0),
    (W("bias_full_mask_ragged", 1, 2, 1, 333, 128, rotary_dim=0, causal=False, seed_id=704), "full", 0.0),
    (W("bias_window_alibi", 1, 4, 4, 640, 128, theta=1e4, window=200, alibi=True, seed_id=705), "full", 0.0),
    (W("bias_minus_inf_entries", 1, 4, 2, 256, 128, theta=1e4, causal=False, seed_id=706), "full", 0.3),
    (W("bias_odd_length_scalar_loads", 1, 2, 2, 259, 64, theta=1e4, seed_id=707), "per_head", 0.0),
]


@pytest.mark.parametrize("w,extent,minf", BIAS_CASES, ids=lambda x: x.name if hasattr(x, "name") else None)
def test_additive_bias(w, extent, minf):
    sb, sh = {"full": (w.B, w.Hq), "per_batch": (w.B, 1), "per_head": (1, w.Hq), "shared": (1, 1)}[extent]
    run(w, bias=bias_of(w, sb, sh, 1, minf))


def test_bias_filled_with_the_alibi_term_matches_the_alibi_kernel():
    w = W("bias_is_alibi", 1, 4, 2, 512, 128, theta=1e4, alibi=True, seed_id=710)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    o_a, l_a = af.fwd(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale)
    ji = (np.arange(w.S)[None, :] - np.arange(w.S)[:, None]).astype(np.float32)
    bias = (w.alibi_slopes()[None, :, None, None] * ji[None, None]).astype(np.float32)
    o_b, l_b = af.fwd_variant(dev["q"], dev["k"], dev["v"], rope, table, af.MaskSpec(causal=True), w.scale,
                              bias=torch.from_numpy(bias).cuda())
    torch.cuda.synchronize()
    assert (o_a.float() - o_b.float()).abs().max().item() <= 8e-3
    assert (l_a - l_b).abs().max().item() <= 1e-3


RELU_CASES = [
    W("relu_causal_gqa", 2, 4, 2, 384, 128, theta=5e5, seed_id=720),
    W("relu_full_d64", 1, 4, 4, 300, 64, theta=1e4, causal=False, seed_id=721),
    W("relu_window_alibi", 1, 4, 2, 640, 128, theta=1e4, window=150, alibi=True, seed_id=722),
    W("relu_norope_ragged", 1, 2, 1, 130, 128, rotary_dim=0, seed_id=723),
]


@pytest.mark.parametrize("w", RELU_CASES, ids=lambda w: w.name)
def test_relu_attention(w):
    run(w, normaliser="relu")


def test_relu_attention_with_bias_and_fp32_output():
    w = W("relu_bias", 1, 4, 2, 400, 128, theta=1e4, seed_id=730)
    run(w, bias=bias_of(w, 1, w.Hq, 2, 0.2), normaliser="relu", out_dtype=torch.float32)


def test_variant_without_extras_is_the_plain_forward_bit_for_bit():
    w = W("variant_plain", 1, 8, 2, 640, 128, theta=5e5, seed_id=740)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    o_a, l_a = af.fwd(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale)
    o_b, l_b = af.fwd_variant(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale)
    torch.cuda.synchronize()
    assert torch.equal(o_a, o_b) and torch.equal(l_a, l_b)


def test_variant_over_block_lists_with_bias():
    w = W("variant_blocks_bias", 1, 4, 2, 640, 128, theta=1e4, causal=False, seed_id=750)
    nb = (w.S + 127) // 128
    active = np.eye(nb, dtype=bool)
    active[:, 0] = True
    active[2, 4] = True
    bias = bias_of(w, 1, 1, 3)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    o, lse = af.fwd_variant(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale, bias=torch.from_numpy(bias).cuda(),
                            blocks=af.BlockMask(active))
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    want_o, want_l = oracle.fwd(t["q"], t["k"], t["v"], theta=w.theta, rotary_dim=w.R, causal=False, scale=w.scale, bias=bias,
                                blocks=active, block_size=128)
    pu.assert_close("blocks + bias O", pu.to_np(o), want_o)
    assert np.abs(pu.to_np(lse) - want_l).max() <= pu.LSE_TOL


def test_variant_argument_errors():
    w = W("variant_errors", 1, 2, 2, 128, 128, rotary_dim=0, seed_id=760)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    bad = torch.zeros((3, 1, w.S, w.S), dtype=torch.float32, device="cuda")     # batch extent neither 1 nor B
    with pytest.raises(af.AttnFuseError) as e:
        af.fwd_variant(dev["q"], dev["k"], dev["v"], af.RopeSpec(), None, af.MaskSpec(), w.scale, bias=bad)
    assert e.value.code == 2
    with pytest.raises(af.AttnFuseError) as e:
        af.fwd_variant(dev["q"], dev["k"], dev["v"], af.RopeSpec(), None, af.MaskSpec(), w.scale, normaliser="relu",
                       blocks=af.BlockMask(np.ones((1, 1), bool)))
    assert e.value.code == 5
