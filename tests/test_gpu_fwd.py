"""GPU parity of the fused forward and of the separate RoPE pass against the fp64 oracle,
element by element on the same seeded inputs, through the C-ABI binding."""
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
    W("norope_dense_1tile", 1, 1, 1, 128, 128, rotary_dim=0, causal=False, seed_id=101),
    W("norope_causal_gqa", 2, 4, 2, 512, 128, rotary_dim=0, seed_id=102),
    W("rope_causal_1tile", 1, 1, 1, 128, 128, theta=1e4, seed_id=103),
    W("rope_causal_gqa4", 1, 8, 2, 640, 128, theta=5e5, seed_id=104),
    W("rope_causal_d64", 2, 4, 4, 384, 64, theta=1e4, seed_id=105),
    W("rope_dense_d64", 1, 2, 1, 300, 64, theta=1e4, causal=False, seed_id=106),
    W("ragged_tail", 1, 4, 1, 333, 128, theta=1e4, seed_id=107),
    W("shorter_than_tile", 1, 2, 2, 37, 128, theta=1e4, seed_id=108),
    W("single_row", 1, 2, 1, 1, 64, theta=1e4, seed_id=109),
    W("window_alibi", 1, 4, 2, 700, 128, theta=1e4, window=200, alibi=True, seed_id=110),
    W("window_small", 1, 2, 2, 520, 128, theta=1e4, window=5, seed_id=111),
    W("window_zero", 1, 2, 2, 260, 64, theta=1e4, window=0, seed_id=112),
    W("window_noncausal", 1, 2, 1, 515, 128, theta=1e4, causal=False, window=130, seed_id=113),
    W("alibi_noncausal", 1, 4, 4, 260, 128, theta=1e4, causal=False, alibi=True, seed_id=114),
    W("partial_rotary", 1, 2, 2, 256, 128, theta=1e4, rotary_dim=64, seed_id=115),
    W("partial_rotary_48_of_64", 1, 2, 2, 200, 64, theta=1e4, rotary_dim=48, seed_id=116),
    W("pos_offset", 1, 2, 1, 384, 128, theta=5e5, pos_offset=1000, seed_id=117),
    W("pos_offset_large", 1, 2, 1, 256, 128, theta=5e5, pos_offset=32768 - 256, sigma=0.5, seed_id=118),
]


def run_case(w, out_dtype=torch.bfloat16, lse_tol=pu.LSE_TOL):
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    # poison outputs: a kernel that skips rows leaves NaNs behind
    o = torch.full((w.B, w.Hq, w.S, w.D), float("nan"), dtype=out_dtype, device="cuda")
    lse = torch.full((w.B, w.Hq, w.S), float("nan"), dtype=torch.float32, device="cuda")
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    af.fwd(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale, out=o, lse=lse)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    want_o, want_l = oracle.run_workload(w, t)
    pu.assert_close(w.name + " O", pu.to_np(o), want_o)
    got_l = pu.to_np(lse)
    assert np.isfinite(got_l).all()
    assert np.abs(got_l - want_l).max() <= lse_tol


@pytest.mark.parametrize("w", SMALL, ids=lambda w: w.name)
def test_forward_small(w):
    run_case(w)


@pytest.mark.parametrize("w", [SMALL[i] for i in (2, 3, 4, 5, 6, 7, 9, 10, 11, 12, 14, 16, 17)] + [synth.CONFIGS[1]],
                         ids=lambda w: w.name)
def test_forward_keys_rotated_in_packed_bf16(w):
    """Optional forward mode: key tiles rotated in packed bf16 arithmetic from TMA-fed tiles of the table's bf16
    copy.  The outputs are held to the same bounds; L gets the output bound, because a row with a single kept
    key has L equal to its one scaled score, which here carries about three bf16 roundings per key element
    (1.1e-2 was measured on such rows at D = 64)."""
    with af.option(af.OPT_FWD_KEYS_BF16, 1):
        run_case(w, lse_tol=2e-2)


ALIBI_CASES = [w for w in SMALL if w.alibi] + [
    W("alibi_gqa_d64", 2, 6, 2, 450, 64, theta=1e4, alibi=True, seed_id=171),
    W("alibi_no_rope_window", 1, 4, 4, 390, 128, rotary_dim=0, window=130, alibi=True, seed_id=172),
    W("alibi_odd_group", 1, 3, 1, 300, 128, theta=1e4, alibi=True, seed_id=173),
]


@pytest.mark.parametrize("w", ALIBI_CASES, ids=lambda w: w.name)
def test_forward_alibi_in_the_softmax_warps(w):
    """ALiBi has two implementations in the forward kernel: by default one more K step of the score product adds
    slope (j - i) (run by every other ALiBi case of this suite); with the option off the softmax warps add it,
    one fused multiply-add per score.  Both are held to the oracle."""
    with af.option(af.OPT_FWD_ALIBI_MMA, 0):
        run_case(w)


@pytest.mark.parametrize("w", ALIBI_CASES, ids=lambda w: w.name)
def test_forward_alibi_by_the_tensor_core(w):
    assert af.get_option(af.OPT_FWD_ALIBI_MMA) == 1   # the default: in the kernels that rotate on chip
    with af.option(af.OPT_FWD_ALIBI_MMA, 2):          # here: also without RoPE
        run_case(w)


@pytest.mark.parametrize("w", SMALL[3:8], ids=lambda w: w.name)
def test_forward_small_one_query_tile_per_cta(w):
    with af.option(af.OPT_FWD_QTILES, 1):
        run_case(w)


@pytest.mark.parametrize("w", [SMALL[i] for i in (1, 3, 4, 6, 9, 12)], ids=lambda w: w.name)
def test_forward_small_row_block_pairs(w):
    """Even GQA groups with head pairing switched off: the two query tiles of a work item are consecutive row
    blocks of one head, with different key ranges."""
    with af.option(af.OPT_FWD_PAIR_HEADS, 0):
        run_case(w)


@pytest.mark.parametrize("w", [SMALL[i] for i in (1, 3, 4, 6, 7, 9, 12, 14, 15, 17)] + [synth.CONFIGS[1]],
                         ids=lambda w: w.name)
def test_forward_hybrid_prerotated_keys(w):
    """Hybrid arm of the fuse-or-not experiment: K rotated once by the RoPE pass into a workspace, Q rotated in
    the kernel.  Held to the oracle like the fused call, and to the fused call itself up to bf16 roundings."""
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S) if w.R > 0 else None
    o, lse = af.fwd_hybrid(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale)
    o_f, lse_f = af.fwd(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    want_o, want_l = oracle.run_workload(w, t)
    pu.assert_close(w.name + " O hybrid", pu.to_np(o), want_o)
    assert np.abs(pu.to_np(lse) - want_l).max() <= pu.LSE_TOL
    assert (o.float() - o_f.float()).abs().max().item() <= 8e-3
    assert (lse - lse_f).abs().max().item() <= 2e-3


def test_forward_hybrid_strided_inputs_and_small_workspace():
    w = W("hybrid_strided", 2, 4, 2, 300, 128, theta=1e4, seed_id=131)
    t = synth.draw_all(w)
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    # K and V as slices of one packed [B, S, 2, Hkv, D] buffer
    kv = torch.empty((w.B, w.S, 2, w.Hkv, w.D), dtype=torch.bfloat16, device="cuda")
    kv[:, :, 0] = pu.to_dev(t["k"]).permute(0, 2, 1, 3)
    kv[:, :, 1] = pu.to_dev(t["v"]).permute(0, 2, 1, 3)
    k = kv[:, :, 0].permute(0, 2, 1, 3)
    v = kv[:, :, 1].permute(0, 2, 1, 3)
    o, _ = af.fwd_hybrid(pu.to_dev(t["q"]), k, v, rope, table, mask, w.scale)
    torch.cuda.synchronize()
    want_o, _ = oracle.run_workload(w, t)
    pu.assert_close("hybrid strided O", pu.to_np(o), want_o)
    with pytest.raises(af.AttnFuseError):
        af.fwd_hybrid(pu.to_dev(t["q"]), k, v, rope, table, mask, w.scale,
                      workspace=torch.empty(1024, dtype=torch.uint8, device="cuda"))


@pytest.mark.parametrize("w", [
    W("host_gqa_chunks", 1, 8, 4, 300, 128, theta=5e5, seed_id=141),                     # 4 chunks of one kv head
    W("host_batches", 9, 4, 2, 200, 64, theta=1e4, seed_id=142),                          # chunks of two batch elements
    W("host_alibi", 2, 8, 4, 260, 128, theta=1e4, window=100, alibi=True, seed_id=143),   # slopes offset per chunk
    W("host_single_chunk", 1, 2, 1, 150, 128, theta=1e4, seed_id=144),
], ids=lambda w: w.name)
def test_forward_from_host_buffers(w):
    """attnfuse_fwd_host: pinned host tensors in and out, the copies and the kernels of consecutive chunks of
    (batch, kv head) units pipelined on internal streams.  Same bounds as the device call, and bit-identical to it."""
    t = synth.draw_all(w)
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    hq, hk, hv = (pu.to_dev(t[k]).cpu().pin_memory() for k in ("q", "k", "v"))
    ho = torch.full(hq.shape, float("nan"), dtype=torch.bfloat16).pin_memory()
    hl = torch.full((w.B, w.Hq, w.S), float("nan"), dtype=torch.float32).pin_memory()
    from paper_2609_13612_b200 import binding
    staging = torch.empty(binding.fwd_host_staging_bytes(w.B, w.Hq, w.Hkv, w.S, w.D), dtype=torch.uint8, device="cuda")
    for _ in range(2):   # a second call reuses the staging buffer behind the first
        af.fwd_host(hq, hk, hv, rope, table, mask, w.scale, ho, hl, staging)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    want_o, want_l = oracle.run_workload(w, t)
    pu.assert_close(w.name + " O from host", pu.to_np(ho), want_o)
    assert np.abs(hl.numpy() - want_l).max() <= pu.LSE_TOL
    o_dev, l_dev = af.fwd(hq.cuda(), hk.cuda(), hv.cuda(), rope, table, mask, w.scale)
    torch.cuda.synchronize()
    assert torch.equal(o_dev.cpu(), ho) and torch.equal(l_dev.cpu(), hl)


def test_forward_fp32_output():
    run_case(W("fp32_out", 1, 4, 2, 300, 128, theta=1e4, seed_id=120), out_dtype=torch.float32)


def test_forward_strided_inputs():
    """q, k, v given as [B,S,H,D] storage viewed as [B,H,S,D] (the layout projection GEMMs produce)."""
    w = W("strided", 2, 4, 2, 260, 128, theta=1e4, seed_id=121)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    perm = {k: v.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3) for k, v in dev.items()}
    assert not perm["q"].is_contiguous()
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    o, lse = af.fwd(perm["q"], perm["k"], perm["v"], rope, table, mask, w.scale)
    o2, lse2 = af.fwd(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale)
    torch.cuda.synchronize()
    assert torch.equal(o, o2) and torch.equal(lse, lse2)


def test_forward_is_deterministic_and_guard_bands_stay_intact():
    w = W("guard", 1, 4, 2, 333, 128, theta=1e4, seed_id=122)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    n = w.B * w.Hq * w.S * w.D
    pad = 4096
    buf = torch.full((n + 2 * pad,), 7.0, dtype=torch.bfloat16, device="cuda")
    o = buf[pad:pad + n].view(w.B, w.Hq, w.S, w.D)
    af.fwd(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale, out=o)
    first = o.clone()
    af.fwd(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale, out=o)
    torch.cuda.synchronize()
    assert torch.equal(first, o)
    assert (buf[:pad] == 7.0).all() and (buf[pad + n:] == 7.0).all()


def test_fused_equals_separate_rope_then_plain_attention():
    """The pre-rotation arm: rotate Q and K with the separate kernel, then run the same
    attention kernel with the rotation switched off."""
    w = W("separate", 1, 8, 2, 640, 128, theta=5e5, seed_id=123)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    qr = af.rope(dev["q"], rope, table)
    kr = af.rope(dev["k"], rope, table)
    o_sep, lse_sep = af.fwd(qr, kr, dev["v"], af.RopeSpec(), None, mask, w.scale)
    o_fus, lse_fus = af.fwd(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale)
    torch.cuda.synchronize()
    # same rounding points (rotated rows rounded to bf16 before the MMA); the fused kernel walks its
    # cos/sin from row to row, so a few bf16 roundings of rotated elements may flip by one ulp
    assert (o_sep.float() - o_fus.float()).abs().max().item() <= 8e-3
    assert (lse_sep - lse_fus).abs().max().item() <= 2e-3
    want_o, _ = oracle.run_workload(w, t)
    pu.assert_close("separate O", pu.to_np(o_sep), want_o)
    pu.assert_close("fused O", pu.to_np(o_fus), want_o)


@pytest.mark.parametrize("R,inverse,D", [(128, False, 128), (64, False, 128), (128, True, 128), (64, False, 64),
                                         (48, True, 64)])
def test_rope_kernel_matches_oracle(R, inverse, D):
    w = W("rope", 2, 5, 5, 301, D, theta=5e5, seed_id=130 + R)
    x = synth.draw(w, "q")
    rs = af.RopeSpec(theta=w.theta, rotary_dim=R, pos_offset=77)
    table = af.rope_table(rs, w.S)
    y = af.rope(pu.to_dev(x), rs, table, inverse=inverse)
    torch.cuda.synchronize()
    want = oracle.rope(x, w.theta, R, 77, inverse=inverse)
    got = pu.to_np(y)
    # output is bf16: half an ulp of the largest magnitude (< 8) is 2^-6
    assert np.abs(got - want).max() <= 2.0 ** -6 + 1e-6
    assert np.abs(got - want).mean() <= 2e-3
    # in place gives the same bits
    xd = pu.to_dev(x)
    af.rope(xd, rs, table, inverse=inverse, out=xd)
    torch.cuda.synchronize()
    assert torch.equal(xd, y)


def test_rope_table_against_fp64_formula():
    rs = af.RopeSpec(theta=500000.0, rotary_dim=128, pos_offset=32768 - 512)
    table = af.rope_table(rs, 512)
    torch.cuda.synchronize()
    pos = rs.pos_offset + np.arange(512)[:, None]
    freq = 500000.0 ** (-2.0 * np.arange(64) / 128)
    assert np.abs(pu.to_np(table[:512, :, 0]) - np.cos(pos * freq)).max() < 1e-7
    assert np.abs(pu.to_np(table[:512, :, 1]) - np.sin(pos * freq)).max() < 1e-7
    assert np.abs(pu.to_np(table[512, :, 0]) - np.cos(16 * freq)).max() < 1e-7  # trailer: stride 16 rows for R = 128
    # the bf16 copy behind the fp32 rows: [64 cos | 64 sin] per position, each the bf16 rounding of the fp32 entry
    raw = table.untyped_storage()
    off = (513 * 64 * 8 + 255) // 256 * 256
    assert raw.nbytes() == off + 512 * 128 * 2
    copy = torch.empty(0, dtype=torch.bfloat16, device=table.device).set_(raw, off // 2, (512, 128))
    assert torch.equal(copy[:, :64], table[:512, :, 0].to(torch.bfloat16))
    assert torch.equal(copy[:, 64:], table[:512, :, 1].to(torch.bfloat16))
    assert np.abs(pu.to_np(copy[:, :64].float()) - np.cos(pos * freq)).max() <= 2.0 ** -9


def test_config1_tiny_and_config2_full():
    for w in synth.CONFIGS[:2]:
        run_case(w)


def test_config3_composed_variant_full():
    """Config 3 at full size (window 1024 + ALiBi): every row of every head against the oracle."""
    w = synth.CONFIGS[2]
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    o, lse = pu.gpu_fwd(w, dev)
    want_o, want_l = oracle.run_workload(w, t)
    got_o, got_l = pu.to_np(o), pu.to_np(lse)
    for h in range(w.Hq):   # per head, so that a failure names the slope it belongs to
        pu.assert_close("c3 O head %d" % h, got_o[:, h], want_o[:, h])
    assert np.abs(got_l - want_l).max() <= pu.LSE_TOL


def test_config4_long_context_sampled_rows():
    """Config 4 at full size: a stratified subset of query rows of every head (first rows, tile
    boundaries, every 509th row, the last rows), each computed one by one by the oracle."""
    w = synth.CONFIGS[3]
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    o, lse = pu.gpu_fwd(w, dev)
    rows = sorted(set([0, 1, 2, 127, 128, 129, 255, 256, 257] + list(range(300, w.S, 509)) +
                      list(range(w.S - 3, w.S))))
    want_o, want_l = oracle.run_workload(w, t, rows=rows)
    idx = torch.tensor(rows, device="cuda")
    pu.assert_close("c4 O", pu.to_np(o[:, :, idx]), want_o)
    assert np.abs(pu.to_np(lse[:, :, idx]) - want_l).max() <= pu.LSE_TOL
