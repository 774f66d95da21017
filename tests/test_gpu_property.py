"""Property-based parity (Section 6.6 of the paper checks its kernels with generated examples across forward and
backward): shapes, GQA groups, rotary widths, position offsets, masks, ALiBi, block lists and workspace sizes are
drawn by hypothesis from a fixed (derandomised) stream, and every example is compared element by element with
the fp64 oracle on the same seeded inputs, at the bounds of the other parity tests plus a relative share of one bf16
ulp of the exact value (parity_util.assert_close_scaled says why).

The kernels branch on many of these parameters - ragged last tiles, head pairs on even groups and row pairs on
odd ones, the rotary widths with a fast path against the generic one, window edges that fall on tile borders,
workspace set-ups of the backward - and the hand-picked cases elsewhere cannot cover their product."""
import numpy as np
import pytest
import torch
from hypothesis import HealthCheck, given, settings, strategies as st

import oracle
import paper_2609_13612_b200 as af
from paper_2609_13612_b200 import synth
import parity_util as pu

pytestmark = pytest.mark.gpu

COMMON = dict(derandomize=True, deadline=None, database=None,
              suppress_health_check=[HealthCheck.too_slow, HealthCheck.data_too_large])


@st.composite
def workloads(draw, backward):
    D = draw(st.sampled_from([64, 128]))
    g = draw(st.sampled_from([1, 2, 3, 4, 8]))
    Hkv = draw(st.integers(1, 2))
    B = draw(st.integers(1, 2))
    # lengths around tile borders, short ones, and ragged ones up to a few tiles
    S = draw(st.one_of(st.sampled_from([1, 127, 128, 129, 255, 256, 257, 384, 512, 640]), st.integers(2, 700)))
    R = draw(st.sampled_from([0, 16, 32, 48, 64, 96, 128]).filter(lambda r: r <= D))
    causal = draw(st.booleans())
    window = draw(st.one_of(st.just(-1), st.sampled_from([0, 1, 127, 128, 129, 256]), st.integers(0, 700)))
    alibi = draw(st.booleans())
    p0 = draw(st.sampled_from([0, 0, 1, 1000, 32768 - 700]))
    theta = draw(st.sampled_from([1.0e4, 5.0e5]))
    sigma = draw(st.sampled_from([0.5, 1.0]))
    seed = draw(st.integers(1000, 1 << 20))
    return synth.Workload("hyp", B, Hkv * g, Hkv, S, D, theta=theta, rotary_dim=R, pos_offset=p0, causal=causal,
                          window=window, alibi=alibi, sigma=sigma, seed_id=seed, backward=backward)


@settings(max_examples=50, **COMMON)
@given(w=workloads(backward=False), f32_out=st.booleans(), hybrid=st.booleans())
def test_forward_examples(w, f32_out, hybrid):
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S) if w.R > 0 else None
    call = af.fwd_hybrid if hybrid else af.fwd
    o, lse = call(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale,
                  out_dtype=torch.float32 if f32_out else torch.bfloat16)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    want_o, want_l = oracle.run_workload(w, t)
    pu.assert_close_scaled("%r O" % (w,), pu.to_np(o), want_o)
    assert np.abs(pu.to_np(lse) - want_l).max() <= pu.LSE_TOL, w


@settings(max_examples=30, **COMMON)
@given(w=workloads(backward=True), tier=st.integers(0, 3), dq_f32=st.booleans())
def test_backward_examples(w, tier, dq_f32):
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S) if w.R > 0 else None
    o, lse = af.fwd(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale)
    # workspace set-ups: delta alone / + rotated-K cache / + rotated-Q cache as well / + dQ accumulator
    n_delta = (w.B * w.Hq * w.S * 4 + 255) // 256 * 256
    n_k = w.B * w.Hkv * w.S * w.D * 2
    n_q = w.B * w.Hq * w.S * w.D * 2
    # (tier 3: room for the fp32 dQ accumulator too - the one-pass sequence where it applies, D = 128)
    ws = torch.empty(n_delta + (n_k if tier >= 1 else 0) + (n_q if tier >= 2 else 0) + (2 * n_q if tier >= 3 else 0),
                     dtype=torch.uint8, device="cuda")
    dq, dk, dv = af.bwd(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale,
                        dq_dtype=torch.float32 if dq_f32 else torch.bfloat16, dkv_dtype=torch.float32, workspace=ws)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    wq, wk, wv = oracle.run_workload(w, t, backward=True)
    # A causal window narrower than the 16 rows that the fp32 first-rows kernel covers makes EVERY row a row with a
    # handful of keys: probabilities are O(1) everywhere, nothing averages the bf16 roundings of P and dS, and the
    # gradients carry them at full size (0.028 measured on dK at window 1).  None of the benchmark configurations is
    # of that kind (the narrowest window is 1024); for generated examples of that kind the stated bound is 4e-2.
    # The same holds for ALiBi WITHOUT a causal mask: the term slope (j - i) grows with j, so every row puts its weight on
    # the last few keys of the sequence: dK and dV of those key rows are sums over ALL g S query rows of terms whose dS
    # (or P) is an O(1) number rounded to bf16, so their error grows like 2^-9 sqrt(g S) |q'| - 0.05 at g S = 1000 -
    # instead of averaging away.  Longer campaigns over other seeds (hypothesis searches for the worst case it can
    # reach) measured up to 0.049 there and nothing above 2e-2 outside these classes.  The paper composes ALiBi with
    # causal only; no benchmark configuration is of this kind.  Stated bound for that class: the common bound plus twice
    # that estimate, 2e-2 + 2 x 2^-9 sqrt(g S) (measured: 0.091 at g S = 2128, where the estimate itself is 0.090).
    tol, mean_tol = pu.MAX_ABS_TOL, pu.MEAN_ABS_TOL
    if 0 <= w.window < 16:      # with or without the causal rule (two-sided: at most 2 W + 1 keys per row)
        tol, mean_tol = 4e-2, 2 * pu.MEAN_ABS_TOL      # nothing averages on any row: the mean error doubles as well
    if not w.causal and w.alibi:
        tol = 2e-2 + 2.0 * 2.0 ** -9 * float(np.sqrt(w.group * w.S))
    pu.assert_close_scaled("%r dQ" % (w,), pu.to_np(dq), wq, max_tol=tol, mean_tol=mean_tol)
    pu.assert_close_scaled("%r dK" % (w,), pu.to_np(dk), wk, max_tol=tol, mean_tol=mean_tol)
    pu.assert_close_scaled("%r dV" % (w,), pu.to_np(dv), wv, max_tol=tol, mean_tol=mean_tol)


@st.composite
def block_patterns(draw, nb):
    """A random set of active 128 x 128 blocks, sometimes with empty row blocks."""
    density = draw(st.sampled_from([0.15, 0.4, 0.8]))
    bits = draw(st.lists(st.floats(0, 1), min_size=nb * nb, max_size=nb * nb))
    a = (np.array(bits).reshape(nb, nb) < density)
    if draw(st.booleans()):
        a |= np.eye(nb, dtype=bool)        # keep the diagonal: no empty rows under a causal mask
    return a


@settings(max_examples=20, **COMMON)
@given(data=st.data())
def test_block_sparse_examples(data):
    D = data.draw(st.sampled_from([64, 128]))
    g = data.draw(st.sampled_from([1, 2, 3, 4]))
    S = data.draw(st.sampled_from([128, 200, 384, 515, 640]))
    causal = data.draw(st.booleans())
    R = data.draw(st.sampled_from([0, 32, 64]))
    seed = data.draw(st.integers(2000, 1 << 20))
    nb = (S + 127) // 128
    active = data.draw(block_patterns(nb))
    w = synth.Workload("hypbs", 1, 2 * g, 2, S, D, theta=1.0e4, rotary_dim=R, causal=causal, seed_id=seed, backward=True)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S) if w.R > 0 else None
    bm = af.BlockMask(active)
    o, lse = af.fwd_blocks(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale, bm)
    dq, dk, dv = af.bwd(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale, blocks=bm)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    kw = dict(theta=w.theta, rotary_dim=w.R, pos_offset=0, causal=causal, window=-1, slopes=None, scale=w.scale)
    want_o, want_l = oracle.fwd(t["q"], t["k"], t["v"], blocks=active, block_size=128, **kw)
    pu.assert_close_scaled("bs O", pu.to_np(o), want_o)
    got_l = pu.to_np(lse)
    fin = np.isfinite(want_l)
    assert np.array_equal(np.isneginf(got_l), np.isneginf(want_l))
    assert np.abs(got_l[fin] - want_l[fin]).max(initial=0.0) <= pu.LSE_TOL
    wq, wk, wv = oracle.bwd(t["q"], t["k"], t["v"], t["do"], blocks=active, block_size=128, **kw)
    # Over block lists there is no fp32 pass for few-key rows (a listed pattern has no "first rows"), and the generated
    # patterns are full of them: under a causal mask the first rows of every row block whose list holds only its
    # diagonal block see a handful of keys.  On such a row P is O(1) and dS = P (dP - delta) is as large as dP itself
    # (|dO . v| reaches 30-40 at D = 128), so its bf16 rounding is up to 2^-9 x 40 = 0.08 per term before the scale c
    # and the sum over the block's rows.  Stated bound for generated block patterns: 1e-1 (campaigns of 2500 examples
    # over other seeds, in which hypothesis searches for the worst case it can reach, measured up to 0.067; the mean
    # error stays at 2-3e-4).
    pu.assert_close_scaled("bs dQ", pu.to_np(dq), wq, max_tol=1e-1)
    pu.assert_close_scaled("bs dK", pu.to_np(dk), wk, max_tol=1e-1)
    pu.assert_close_scaled("bs dV", pu.to_np(dv), wv, max_tol=1e-1)


@settings(max_examples=20, **COMMON)
@given(w=workloads(backward=True), extent=st.sampled_from(["full", "per_batch", "per_head", "shared"]),
       minus_inf=st.sampled_from([0.0, 0.0, 0.25]))
def test_additive_bias_examples(w, extent, minus_inf):
    """Forward and backward of `additive_bias` composed with whatever else the example draws (Section 3.1)."""
    sb, sh = {"full": (w.B, w.Hq), "per_batch": (w.B, 1), "per_head": (1, w.Hq), "shared": (1, 1)}[extent]
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([synth.BASE_SEED, w.seed_id, 11])))
    bias = (0.5 * rng.standard_normal((sb, sh, w.S, w.S))).astype(np.float32)
    if minus_inf > 0:
        drop = rng.random(bias.shape) < minus_inf
        drop[..., np.arange(w.S), np.arange(w.S)] = False      # keep the diagonal: no empty rows
        bias[drop] = -np.inf
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S) if w.R > 0 else None
    bias_dev = torch.from_numpy(bias).cuda()
    o, lse = af.fwd_variant(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale, bias=bias_dev)
    dq, dk, dv = af.bwd_variant(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale, bias=bias_dev,
                                dq_dtype=torch.float32)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    kw = dict(theta=w.theta, rotary_dim=w.R, pos_offset=w.pos_offset, causal=w.causal, window=w.window,
              slopes=w.alibi_slopes(), scale=w.scale, bias=bias)
    want_o, want_l = oracle.fwd(t["q"], t["k"], t["v"], **kw)
    pu.assert_close_scaled("%r bias O" % (w,), pu.to_np(o), want_o)
    assert np.abs(pu.to_np(lse) - want_l).max() <= pu.LSE_TOL, w
    wq, wk, wv = oracle.bwd(t["q"], t["k"], t["v"], t["do"], **kw)
    # The variant backward has no fp32 pass over the first query rows, and the drawn examples are full of rows whose
    # probability mass sits on a handful of keys (causal first rows, -inf entries, non-causal ALiBi rows that collapse
    # onto the last keys): those rows carry the bf16 roundings of P and dS at full size, the case the plain backward
    # treats separately.  Stated bound for generated examples of this entry point: 4e-2 (measured worst 0.021-0.03), and
    # plus 2 x 2^-9 sqrt(g S) for ALiBi without a causal mask, where every row collapses onto the last keys and their
    # dK and dV sum un-averaged roundings over all g S query rows (see test_backward_examples; measured up to 0.097).
    tol = 4e-2 + 2.0 * 2.0 ** -9 * float(np.sqrt(w.group * w.S)) if (not w.causal and w.alibi) else 4e-2
    pu.assert_close_scaled("%r bias dQ" % (w,), pu.to_np(dq), wq, max_tol=tol)
    pu.assert_close_scaled("%r bias dK" % (w,), pu.to_np(dk), wk, max_tol=tol)
    pu.assert_close_scaled("%r bias dV" % (w,), pu.to_np(dv), wv, max_tol=tol)
