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
        # the row statistic of the ReLU normaliser is n_i, the number of kept pairs with a finite score: an integer,
        # compared exactly with a count written out here from the mask definition
        assert want_l is None
        assert np.array_equal(pu.to_np(lse), kept_counts(w, bias))
    return o


def kept_counts(w, bias):
    """n_i[b, h, i]: pairs (i, j) that the mask keeps and whose bias is finite."""
    i = np.arange(w.S)[:, None]
    j = np.arange(w.S)[None, :]
    keep = np.ones((w.S, w.S), dtype=bool)
    if w.causal:
        keep &= j <= i
        if w.window >= 0:
            keep &= i - j <= w.window
    elif w.window >= 0:
        keep &= np.abs(i - j) <= w.window
    keep = np.broadcast_to(keep, (w.B, w.Hq, w.S, w.S)).copy()
    if bias is not None:
        keep &= np.isfinite(np.broadcast_to(bias, keep.shape))
    return keep.sum(-1).astype(np.float32)


def run_bwd(w, bias=None, normaliser="softmax", max_tol=pu.MAX_ABS_TOL):
    """Forward and backward of the same variant through the C-ABI, gradients against the oracle."""
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S) if w.R > 0 else None
    bias_dev = torch.from_numpy(bias).cuda() if bias is not None else None
    o, lse = af.fwd_variant(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale, bias=bias_dev, normaliser=normaliser)
    dq, dk, dv = af.bwd_variant(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale, bias=bias_dev,
                                normaliser=normaliser, dq_dtype=torch.float32)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    wq, wk, wv = oracle.bwd(t["q"], t["k"], t["v"], t["do"], theta=w.theta, rotary_dim=w.R, pos_offset=w.pos_offset,
                            causal=w.causal, window=w.window, slopes=w.alibi_slopes(), scale=w.scale, bias=bias,
                            normaliser=normaliser)
    if normaliser == "softmax":
        for name, got, want in (("dQ", dq, wq), ("dK", dk, wk), ("dV", dv, wv)):
            pu.assert_close("%s %s (%s)" % (w.name, name, normaliser), pu.to_np(got), want, max_tol=max_tol)
        return
    # ReLU: dS_ij = [s_ij > 0] dP_ij / n_i is discontinuous in the score.  Where |s_ij| is within the score error of
    # the bf16 path (rotated q', k' rounded to bf16: up to ~1e-2 on these sizes) the two sides may take the decision
    # differently, and either decision is a valid gradient of the rounded problem.  Such pairs are found here from
    # the definition, and the rows of dQ and dK that they touch get the size of their contribution as slack; every
    # other element, and the mean over all elements, is held to the stated bounds.  dV does not see the decision.
    slack_q, slack_k = relu_decision_slack(w, t, bias, eps=1e-2)
    pu.assert_close("%s dV (relu)" % w.name, pu.to_np(dv), wv, max_tol=max_tol)
    for name, got, want, slack in (("dQ", dq, wq, slack_q), ("dK", dk, wk, slack_k)):
        d = np.abs(pu.to_np(got) - want)
        assert np.isfinite(d).all()
        assert d.mean() <= pu.MEAN_ABS_TOL, "%s %s: mean abs %.4g" % (w.name, name, d.mean())
        over = d - (max_tol + slack[..., None])
        assert over.max() <= 0, "%s %s: %.4g beyond bound + slack" % (w.name, name, over.max())
        # the decision differs for a handful of pairs only: elements beyond the plain bound stay rare
        frac = (d > max_tol).mean()
        assert frac <= 2e-3, "%s %s: %.3g of the elements beyond %g" % (w.name, name, frac, max_tol)


def relu_decision_slack(w, t, bias, eps):
    """Per query row (for dQ) and per key row (for dK): the largest change of a gradient element if every kept pair
    with |s_ij| < eps took the other decision of [s_ij > 0].  Plain numpy from the definitions, fp64."""
    q = oracle.rope(t["q"], w.theta, w.R, w.pos_offset) if w.R > 0 else np.asarray(t["q"], np.float64)
    k = oracle.rope(t["k"], w.theta, w.R, w.pos_offset) if w.R > 0 else np.asarray(t["k"], np.float64)
    v, do = np.asarray(t["v"], np.float64), np.asarray(t["do"], np.float64)
    g = w.group
    n = kept_counts(w, bias).astype(np.float64)
    ii, jj = np.arange(w.S)[:, None], np.arange(w.S)[None, :]
    keep = np.ones((w.S, w.S), dtype=bool)
    if w.causal:
        keep &= jj <= ii
        if w.window >= 0:
            keep &= ii - jj <= w.window
    elif w.window >= 0:
        keep &= np.abs(ii - jj) <= w.window
    slopes = w.alibi_slopes()
    slack_q = np.zeros((w.B, w.Hq, w.S))
    slack_k = np.zeros((w.B, w.Hkv, w.S))
    for b in range(w.B):
        for h in range(w.Hq):
            hk = h // g
            s = w.scale * q[b, h] @ k[b, hk].T
            if slopes is not None:
                s = s + slopes[h] * (jj - ii)
            kp = keep.copy()
            if bias is not None:
                bb = np.broadcast_to(bias, (w.B, w.Hq, w.S, w.S))[b, h].astype(np.float64)
                kp &= np.isfinite(bb)
                s = s + np.where(np.isfinite(bb), bb, 0.0)
            amb = kp & (np.abs(s) < eps)
            dp = np.abs(do[b, h] @ v[b, hk].T) / np.maximum(n[b, h], 1.0)[:, None] * amb
            # the rotation back mixes a column with its partner: twice the largest element bounds both
            slack_q[b, h] = 2.0 * w.scale * dp @ np.abs(k[b, hk]).max(-1)
            slack_k[b, hk] += 2.0 * w.scale * dp.T @ np.abs(q[b, h]).max(-1)
    return slack_q, slack_k


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


BWD_BIAS_CASES = [
    (W("bwd_bias_causal_gqa", 2, 4, 2, 384, 128, theta=5e5, backward=True, seed_id=770), "full", 0.0),
    (W("bwd_bias_shared_d64", 1, 6, 2, 515, 64, theta=1e4, backward=True, seed_id=771), "shared", 0.0),
    (W("bwd_bias_full_mask_norope", 1, 2, 1, 333, 128, rotary_dim=0, causal=False, backward=True, seed_id=772), "full", 0.0),
    (W("bwd_bias_window_alibi", 1, 4, 4, 640, 128, theta=1e4, window=200, alibi=True, backward=True, seed_id=773), "per_head", 0.0),
    (W("bwd_bias_minus_inf", 1, 4, 2, 256, 128, theta=1e4, causal=False, backward=True, seed_id=774), "per_batch", 0.3),
]


@pytest.mark.parametrize("w,extent,minf", BWD_BIAS_CASES, ids=lambda x: x.name if hasattr(x, "name") else None)
def test_additive_bias_backward(w, extent, minf):
    sb, sh = {"full": (w.B, w.Hq), "per_batch": (w.B, 1), "per_head": (1, w.Hq), "shared": (1, 1)}[extent]
    run_bwd(w, bias=bias_of(w, sb, sh, 4, minf))


BWD_RELU_CASES = [
    W("bwd_relu_causal_gqa", 2, 4, 2, 384, 128, theta=5e5, backward=True, seed_id=780),
    W("bwd_relu_full_d64", 1, 4, 4, 300, 64, theta=1e4, causal=False, backward=True, seed_id=781),
    W("bwd_relu_window_alibi", 1, 4, 2, 640, 128, theta=1e4, window=150, alibi=True, backward=True, seed_id=782),
    W("bwd_relu_norope_ragged", 1, 2, 1, 130, 128, rotary_dim=0, backward=True, seed_id=783),
]


@pytest.mark.parametrize("w", BWD_RELU_CASES, ids=lambda w: w.name)
def test_relu_attention_backward(w):
    # the ReLU normaliser has no sum that averages the score error (see `run`): the bound of its forward
    run_bwd(w, normaliser="relu", max_tol=6e-2)


def test_relu_attention_backward_with_bias():
    w = W("bwd_relu_bias", 1, 4, 2, 400, 128, theta=1e4, backward=True, seed_id=784)
    run_bwd(w, bias=bias_of(w, 1, w.Hq, 5, 0.2), normaliser="relu", max_tol=6e-2)


def test_backward_variant_without_extras_is_the_plain_backward():
    w = W("bwd_variant_plain", 1, 8, 2, 640, 128, theta=5e5, backward=True, seed_id=785)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    o, lse = af.fwd(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale)
    with af.option(af.OPT_BWD_ONEPASS, 0):   # the two-kernel sequence is bit-reproducible
        a = af.bwd(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale)
        b = af.bwd_variant(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale)
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        assert torch.equal(x, y)


def test_backward_variant_argument_errors():
    w = W("bwd_variant_errors", 1, 2, 2, 256, 128, theta=1e4, backward=True, seed_id=786)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    bias = torch.zeros((1, 1, w.S, w.S), dtype=torch.float32, device="cuda")
    o, lse = af.fwd_variant(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale, bias=bias)
    with pytest.raises(af.AttnFuseError) as e:      # extras over block lists are not built
        af.bwd_variant(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale, bias=bias,
                       blocks=af.BlockMask(np.ones((2, 2), bool)))
    assert e.value.code == 5
    small = torch.empty(w.B * w.Hq * w.S * 4 + 256, dtype=torch.uint8, device="cuda")   # delta only: no room for the caches
    with pytest.raises(af.AttnFuseError) as e:
        af.bwd_variant(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale, bias=bias, workspace=small)
    assert e.value.code == 6
