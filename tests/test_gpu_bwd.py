"""GPU parity of the fused backward (dQ, dK, dV with the inverse rotation fused) against the
fp64 oracle, element by element on the same seeded inputs, through the C-ABI binding."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_13612_b200 as af
from paper_2609_13612_b200 import synth
import parity_util as pu

pytestmark = pytest.mark.gpu
W = synth.Workload

SMALL = [
    W("norope_dense_1tile", 1, 1, 1, 128, 128, rotary_dim=0, causal=False, backward=True, seed_id=201),
    W("norope_causal_2tile", 1, 2, 1, 256, 128, rotary_dim=0, backward=True, seed_id=202),
    W("rope_causal_1tile", 1, 1, 1, 128, 128, theta=1e4, backward=True, seed_id=203),
    W("rope_causal_gqa4", 1, 8, 2, 640, 128, theta=5e5, backward=True, seed_id=204),
    W("rope_causal_d64", 2, 4, 4, 384, 64, theta=1e4, backward=True, seed_id=205),
    W("ragged_tail", 1, 4, 1, 333, 128, theta=1e4, backward=True, seed_id=206),
    W("shorter_than_tile", 1, 2, 2, 37, 128, theta=1e4, backward=True, seed_id=207),
    W("single_row", 1, 2, 1, 1, 64, theta=1e4, backward=True, seed_id=208),
    W("window_alibi", 1, 4, 2, 700, 128, theta=1e4, window=200, alibi=True, backward=True, seed_id=209),
    W("window_noncausal", 1, 2, 1, 515, 128, theta=1e4, causal=False, window=130, backward=True, seed_id=210),
    W("partial_rotary", 1, 2, 2, 256, 128, theta=1e4, rotary_dim=64, backward=True, seed_id=211),
    W("partial_rotary_48_of_64", 1, 2, 2, 200, 64, theta=1e4, rotary_dim=48, backward=True, seed_id=212),
    W("pos_offset", 1, 2, 1, 384, 128, theta=5e5, pos_offset=1000, backward=True, seed_id=213),
    W("dense_rope_d64", 1, 2, 1, 300, 64, theta=1e4, causal=False, backward=True, seed_id=214),
]


def run_case(w, dq_dtype=torch.bfloat16, dkv_dtype=torch.float32):
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    o, lse = pu.gpu_fwd(w, dev)
    dq, dk, dv = pu.gpu_bwd(w, dev, o, lse, dq_dtype=dq_dtype, dkv_dtype=dkv_dtype)
    want = oracle.run_workload(w, t, backward=True)
    for name, got, ref in zip(("dQ", "dK", "dV"), (dq, dk, dv), want):
        pu.assert_close("%s %s" % (w.name, name), pu.to_np(got), ref)


@pytest.mark.parametrize("w", SMALL, ids=lambda w: w.name)
def test_backward_small(w):
    run_case(w)


def test_backward_fp32_dq_and_bf16_dkv_outputs():
    w = W("dtypes", 1, 4, 2, 300, 128, theta=1e4, backward=True, sigma=0.5, seed_id=220)
    run_case(w, dq_dtype=torch.float32, dkv_dtype=torch.float32)
    run_case(w, dq_dtype=torch.bfloat16, dkv_dtype=torch.bfloat16)


def test_backward_zero_upstream_gradient_and_determinism():
    w = W("zero_do", 1, 4, 2, 300, 128, theta=1e4, backward=True, seed_id=221)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    o, lse = pu.gpu_fwd(w, dev)
    # two-kernel sequence: every output is bit-reproducible
    with af.option(af.OPT_BWD_ONEPASS, 0):
        a = pu.gpu_bwd(w, dev, o, lse)
        b = pu.gpu_bwd(w, dev, o, lse)
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    # one-pass sequence (the default here: D = 128, full workspace): dK and dV are reproducible, the fp32
    # reductions of dQ in global memory may land in another order
    c = pu.gpu_bwd(w, dev, o, lse)
    d = pu.gpu_bwd(w, dev, o, lse)
    assert torch.equal(c[1], d[1]) and torch.equal(c[2], d[2])
    assert (c[0].float() - d[0].float()).abs().max().item() <= 2.0 ** -7 * c[0].float().abs().max().item()
    dev["do"] = torch.zeros_like(dev["do"])
    for g in pu.gpu_bwd(w, dev, o, lse):
        assert not g.any()
    with af.option(af.OPT_BWD_ONEPASS, 0):
        for g in pu.gpu_bwd(w, dev, o, lse):
            assert not g.any()


def test_backward_strided_inputs():
    w = W("strided", 2, 4, 2, 260, 128, theta=1e4, backward=True, seed_id=222)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    o, lse = pu.gpu_fwd(w, dev)
    ref = pu.gpu_bwd(w, dev, o, lse)
    perm = dict(dev)
    for k in ("q", "k", "v"):
        perm[k] = dev[k].permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    got = pu.gpu_bwd(w, perm, o, lse)
    assert torch.equal(ref[1], got[1]) and torch.equal(ref[2], got[2])
    assert (ref[0].float() - got[0].float()).abs().max().item() <= 2.0 ** -7 * ref[0].float().abs().max().item()
    with af.option(af.OPT_BWD_ONEPASS, 0):
        ref = pu.gpu_bwd(w, dev, o, lse)
        got = pu.gpu_bwd(w, perm, o, lse)
    for x, y in zip(ref, got):
        assert torch.equal(x, y)


def test_backward_workspace_too_small_is_an_error():
    w = W("ws", 1, 2, 1, 128, 128, theta=1e4, backward=True, seed_id=223)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    o, lse = pu.gpu_fwd(w, dev)
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    with pytest.raises(af.AttnFuseError) as e:
        af.bwd(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale,
               workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.code == 6


def test_config5_training_shape_full():
    """Full-size config 5 in the launch configuration the bench times: O, L, dQ, dK and dV of every
    (batch, head) against the oracle."""
    w = synth.CONFIGS[4]
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    o, lse = pu.gpu_fwd(w, dev)
    dq, dk, dv = pu.gpu_bwd(w, dev, o, lse)
    want_o, want_l = oracle.run_workload(w, t)
    pu.assert_close("c5 O", pu.to_np(o), want_o)
    assert np.abs(pu.to_np(lse) - want_l).max() <= pu.LSE_TOL
    wq, wk, wv = oracle.run_workload(w, t, backward=True)
    pu.assert_close("c5 dQ", pu.to_np(dq), wq)
    pu.assert_close("c5 dK", pu.to_np(dk), wk)
    pu.assert_close("c5 dV", pu.to_np(dv), wv)


def test_backward_workspace_tiers_give_the_same_result():
    """Set-ups by workspace size: the one-pass sequence (both caches and the fp32 dQ accumulator), delta + K' cache +
    Q' cache (nothing rotated in the dK/dV loop), delta + K' cache (the dQ kernel streams cached K'), delta alone
    (both kernels rotate on chip).  All match the oracle and agree with one another up to a few bf16 roundings."""
    w = W("ws_tiers", 2, 4, 2, 515, 128, theta=5e5, backward=True, seed_id=224)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    o, lse = pu.gpu_fwd(w, dev)
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    n_delta = (w.B * w.Hq * w.S * 4 + 255) // 256 * 256
    n_k = w.B * w.Hkv * w.S * w.D * 2
    n_q = w.B * w.Hq * w.S * w.D * 2
    assert af.bwd_workspace_bytes(w.B, w.Hq, w.Hkv, w.S, w.D, onepass=False) == n_delta + n_k + n_q
    assert af.bwd_workspace_bytes(w.B, w.Hq, w.Hkv, w.S, w.D) == n_delta + n_k + 3 * n_q
    onepass = af.bwd(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale)
    full_ws = torch.empty(n_delta + n_k + n_q, dtype=torch.uint8, device="cuda")
    full = af.bwd(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale, workspace=full_ws)
    mid_ws = torch.empty(n_delta + n_k, dtype=torch.uint8, device="cuda")
    mid = af.bwd(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale, workspace=mid_ws)
    small_ws = torch.empty(n_delta, dtype=torch.uint8, device="cuda")
    small = af.bwd(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale, workspace=small_ws)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    # with or without the K' cache dK and dV come from the same kernel on the same rotated rows
    assert torch.equal(mid[1], small[1]) and torch.equal(mid[2], small[2])
    # elsewhere cos/sin are walked over different runs of rows (or read from the table), so a few bf16
    # roundings of rotated rows may differ by one ulp
    for a, b in ((onepass, full), (full, mid), (mid, small)):
        for x, y in zip(a, b):
            assert (x.float() - y.float()).abs().max().item() <= 1e-2
    want = oracle.run_workload(w, t, backward=True)
    for res in (onepass, full, mid, small):
        for name, got, ref in zip(("dQ", "dK", "dV"), res, want):
            pu.assert_close("%s %s" % (w.name, name), pu.to_np(got), ref)


def _check_units(w, units, t, o, lse, grads, tag):
    """Oracle forward + backward on whole (batch, kv head) units of a larger workload."""
    dq, dk, dv = grads
    g = w.group
    slopes = w.alibi_slopes()
    for b, hk in units:
        hs = slice(hk * g, (hk + 1) * g)
        kw = dict(theta=w.theta, rotary_dim=w.R, pos_offset=w.pos_offset, causal=w.causal, window=w.window,
                  slopes=None if slopes is None else slopes[hs], scale=w.scale)
        q, k, v, do = t["q"][b:b + 1, hs], t["k"][b:b + 1, hk:hk + 1], t["v"][b:b + 1, hk:hk + 1], t["do"][b:b + 1, hs]
        want_o, want_l = oracle.fwd(q, k, v, **kw)
        pu.assert_close(tag + " O", pu.to_np(o[b:b + 1, hs]), want_o)
        assert np.abs(pu.to_np(lse[b:b + 1, hs]) - want_l).max() <= pu.LSE_TOL
        wq, wk, wv = oracle.bwd(q, k, v, do, **kw)
        pu.assert_close(tag + " dQ", pu.to_np(dq[b:b + 1, hs]), wq)
        pu.assert_close(tag + " dK", pu.to_np(dk[b:b + 1, hk:hk + 1]), wk)
        pu.assert_close(tag + " dV", pu.to_np(dv[b:b + 1, hk:hk + 1]), wv)


def test_gpt2_small_geometry_d64_forward_and_backward_sampled_units():
    """The geometry of Section 5's single-GPU tables (B = 4, 12 heads, D = 64), RoPE + causal, at N = 4096."""
    w = W("gpt2_small_d64", 4, 12, 12, 4096, 64, theta=1e4, backward=True, seed_id=230)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    o, lse = pu.gpu_fwd(w, dev)
    grads = pu.gpu_bwd(w, dev, o, lse)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    _check_units(w, ((0, 0), (3, 11)), t, o, lse, grads, "gpt2-small")


def test_composed_window_alibi_backward_sampled_units():
    """Config 3's composed variant (RoPE + causal + window 1024 + ALiBi) through the backward at S = 8192:
    steep and shallow slopes, both kept-interval edges of the window in many tiles.  With the steepest slope a
    row attends to about three keys, nothing averages out and |dQ| reaches 8: the gradient is taken in fp32,
    since bf16 output rounding alone (half an ulp is 0.016 in [4, 8)) would use up the 2e-2 bound."""
    c3 = synth.CONFIGS[2]
    w = W("c3_bwd", 1, c3.Hq, c3.Hkv, c3.S, c3.D, theta=c3.theta, window=c3.window, alibi=True, backward=True, seed_id=231)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    o, lse = pu.gpu_fwd(w, dev)
    grads = pu.gpu_bwd(w, dev, o, lse, dq_dtype=torch.float32)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    _check_units(w, ((0, 0), (0, w.Hkv - 1)), t, o, lse, grads, "c3 backward")


def test_partial_rotary_at_scale_sampled_units():
    """Rotary dimension 64 of D = 128 (the rest of each row passes through) with GQA at S = 2048."""
    w = W("partial_rotary_2k", 2, 8, 2, 2048, 128, theta=5e5, rotary_dim=64, backward=True, seed_id=232)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    o, lse = pu.gpu_fwd(w, dev)
    grads = pu.gpu_bwd(w, dev, o, lse)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    _check_units(w, ((1, 1),), t, o, lse, grads, "partial rotary")


@pytest.mark.parametrize("mode", [0, 2], ids=["two_kernel", "one_pass"])
def test_both_backward_sequences_on_long_rows_sampled_units(mode):
    """S = 4096 with GQA (16.5 kept key tiles per query tile on average: left to itself the library takes the
    two-kernel sequence here) with either sequence forced, full one-pass workspace in both runs."""
    w = W("long_rows_%d" % mode, 1, 8, 2, 4096, 128, theta=5e5, backward=True, seed_id=233)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    o, lse = pu.gpu_fwd(w, dev)
    with af.option(af.OPT_BWD_ONEPASS, mode):
        grads = pu.gpu_bwd(w, dev, o, lse)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    _check_units(w, ((0, 1),), t, o, lse, grads, "long rows")
