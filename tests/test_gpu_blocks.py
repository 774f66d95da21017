"""GPU parity of block-sparse attention (Section 4.3): the kernels walk index lists of active 128 x 128
blocks; the oracle applies the same block matrix on top of the element mask."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_13612_b200 as af
from paper_2609_13612_b200 import synth
import parity_util as pu

pytestmark = pytest.mark.gpu
W = synth.Workload


def bigbird_blocks(nb, window=1, n_global=1, n_random=1, seed=0, causal=False):
    """BigBird-like pattern over blocks: a band of `window` blocks each side, `n_global` leading global
    block rows/columns and `n_random` random blocks per row (seeded)."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([20260913, 900, seed])))
    a = np.zeros((nb, nb), dtype=bool)
    for i in range(nb):
        a[i, max(0, i - window):min(nb, i + window + 1)] = True
        a[i, rng.integers(0, nb, size=n_random)] = True
    a[:n_global, :] = True
    a[:, :n_global] = True
    if causal:
        a &= np.tril(np.ones((nb, nb), dtype=bool))
    return a


def run_fwd(w, active, out_dtype=torch.bfloat16):
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S) if w.R > 0 else None
    bm = af.BlockMask(active)
    o, lse = af.fwd_blocks(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale, bm, out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    want_o, want_l = oracle.fwd(t["q"], t["k"], t["v"], theta=w.theta, rotary_dim=w.R, pos_offset=w.pos_offset,
                                causal=w.causal, window=w.window, slopes=w.alibi_slopes(), scale=w.scale,
                                blocks=active, block_size=128)
    pu.assert_close(w.name + " O", pu.to_np(o), want_o)
    got_l = pu.to_np(lse)
    fin = np.isfinite(want_l)
    assert np.array_equal(np.isneginf(got_l), np.isneginf(want_l))
    assert np.abs(got_l[fin] - want_l[fin]).max(initial=0.0) <= pu.LSE_TOL
    return t, dev, o, lse, bm


FWD_CASES = [
    (W("bs_dense_pattern", 1, 4, 2, 512, 128, theta=1e4, seed_id=401), lambda nb: np.ones((nb, nb), bool)),
    (W("bs_block_diagonal_noncausal", 1, 4, 2, 640, 128, theta=1e4, causal=False, seed_id=402), lambda nb: np.eye(nb, dtype=bool)),
    (W("bs_bigbird_noncausal", 2, 4, 2, 1024, 128, theta=5e5, causal=False, seed_id=403), lambda nb: bigbird_blocks(nb, seed=1)),
    (W("bs_bigbird_causal", 1, 8, 2, 1100, 128, theta=5e5, seed_id=404), lambda nb: bigbird_blocks(nb, seed=2, causal=True)),
    (W("bs_unsorted_free_lists_d64", 1, 4, 4, 700, 64, theta=1e4, causal=False, seed_id=405), lambda nb: bigbird_blocks(nb, seed=3)),
    (W("bs_odd_group_one_head_per_cta", 1, 3, 1, 600, 128, theta=1e4, causal=False, seed_id=406), lambda nb: bigbird_blocks(nb, seed=4)),
    (W("bs_norope_window_alibi", 1, 4, 2, 900, 128, rotary_dim=0, window=300, alibi=True, seed_id=407), lambda nb: np.tril(np.ones((nb, nb), bool))),
    (W("bs_partial_rotary", 1, 2, 2, 512, 128, theta=1e4, rotary_dim=64, causal=False, seed_id=408), lambda nb: bigbird_blocks(nb, seed=5)),
]


@pytest.mark.parametrize("w,pattern", FWD_CASES, ids=lambda x: x.name if hasattr(x, "name") else "")
def test_block_sparse_forward(w, pattern):
    run_fwd(w, pattern((w.S + 127) // 128))


def test_block_sparse_row_blocks_without_active_blocks_give_zero_rows():
    w = W("bs_empty_rows", 1, 4, 2, 512, 128, theta=1e4, causal=False, seed_id=410)
    a = np.zeros((4, 4), dtype=bool)
    a[0, 1] = a[2, 0] = a[2, 3] = True          # row blocks 1 and 3 have nothing
    t, dev, o, lse, _ = run_fwd(w, a)
    assert torch.all(o[:, :, 128:256] == 0) and torch.all(torch.isneginf(lse[:, :, 128:256]))


def test_block_sparse_row_pairs_of_one_head():
    """Odd GQA group: a CTA takes the row blocks 2r and 2r + 1 of one head and walks the union of their lists.  An odd
    number of row blocks, a row block without blocks inside a pair, a pair without any block, causal + window + ALiBi."""
    w = W("bs_rowpair_mixed", 2, 3, 3, 1100, 128, theta=1e4, window=500, alibi=True, seed_id=412)   # 9 row blocks
    nb = 9
    a = np.tril(bigbird_blocks(nb, seed=7, causal=True))
    a[3, :] = False           # row block 3 (second of pair 1) has nothing
    a[6, :] = a[7, :] = False   # pair 3 has nothing
    t, dev, o, lse, _ = run_fwd(w, a)
    for r in (3, 6, 7):
        assert torch.all(o[:, :, 128 * r:128 * (r + 1)] == 0) and torch.all(torch.isneginf(lse[:, :, 128 * r:128 * (r + 1)]))


@pytest.mark.parametrize("w,pattern", [FWD_CASES[4], FWD_CASES[5]], ids=lambda x: x.name if hasattr(x, "name") else "")
def test_block_sparse_forward_one_row_block_per_cta(w, pattern):
    """The same odd-group cases without the pair lists (one query tile per CTA)."""
    with af.option(af.OPT_BS_ROWPAIR, 0):
        run_fwd(w, pattern((w.S + 127) // 128))


def test_block_sparse_all_active_equals_the_dense_kernel():
    w = W("bs_vs_dense", 1, 4, 2, 768, 128, theta=5e5, seed_id=411)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    # causal: list exactly the tiles the dense kernel visits (lower triangle of blocks)
    bm = af.BlockMask(np.tril(np.ones((6, 6), bool)))
    o1, l1 = af.fwd_blocks(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale, bm)
    o2, l2 = af.fwd(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale)
    # the same arithmetic except that cos/sin are read from the table for every tile instead of walked on
    assert (o1.float() - o2.float()).abs().max().item() <= 8e-3
    assert (l1 - l2).abs().max().item() <= 1e-3


def run_bwd(w, active, workspace_tier=2, dq_dtype=torch.bfloat16):
    t, dev, o, lse, bm = run_fwd(w, active)
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S) if w.R > 0 else None
    n_delta = (w.B * w.Hq * w.S * 4 + 255) // 256 * 256
    # tier 3: room for the fp32 dQ accumulator as well, and the one-pass sequence forced (over block lists it is the
    # default only at D = 64)
    n_ws = n_delta + (w.B * w.Hkv * w.S * w.D * 2 if workspace_tier >= 1 else 0) + \
        (w.B * w.Hq * w.S * w.D * 2 if workspace_tier >= 2 else 0) + (w.B * w.Hq * w.S * w.D * 4 if workspace_tier >= 3 else 0)
    ws = torch.empty(n_ws, dtype=torch.uint8, device="cuda")
    with af.option(af.OPT_BWD_ONEPASS, 2 if workspace_tier >= 3 else 0):
        dq, dk, dv = af.bwd(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale, workspace=ws,
                            blocks=bm, dq_dtype=dq_dtype)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    want = oracle.bwd(t["q"], t["k"], t["v"], t["do"], theta=w.theta, rotary_dim=w.R, pos_offset=w.pos_offset,
                      causal=w.causal, window=w.window, slopes=w.alibi_slopes(), scale=w.scale, blocks=active,
                      block_size=128)
    for name, got, ref in zip(("dQ", "dK", "dV"), (dq, dk, dv), want):
        pu.assert_close("%s %s" % (w.name, name), pu.to_np(got), ref)


BWD_CASES = [
    (W("bsb_dense_pattern", 1, 4, 2, 512, 128, theta=1e4, backward=True, seed_id=421), lambda nb: np.tril(np.ones((nb, nb), bool)), 2),
    (W("bsb_bigbird_noncausal", 2, 4, 2, 1024, 128, theta=5e5, causal=False, backward=True, seed_id=422), lambda nb: bigbird_blocks(nb, seed=11), 2),
    (W("bsb_bigbird_causal_gqa4", 1, 8, 2, 1100, 128, theta=5e5, backward=True, seed_id=423), lambda nb: bigbird_blocks(nb, seed=12, causal=True), 2),
    (W("bsb_bigbird_k_cache_only", 1, 4, 2, 900, 128, theta=1e4, causal=False, backward=True, seed_id=424), lambda nb: bigbird_blocks(nb, seed=13), 1),
    (W("bsb_bigbird_no_cache", 1, 4, 2, 900, 128, theta=1e4, causal=False, backward=True, seed_id=425), lambda nb: bigbird_blocks(nb, seed=14), 0),
    (W("bsb_d64_norope", 1, 4, 4, 700, 64, rotary_dim=0, causal=False, backward=True, seed_id=426), lambda nb: bigbird_blocks(nb, seed=15), 2),
    (W("bsb_window_alibi", 1, 4, 2, 900, 128, theta=1e4, window=300, alibi=True, backward=True, seed_id=427), lambda nb: np.tril(np.ones((nb, nb), bool)), 2),
    (W("bsb_onepass_bigbird_d64", 2, 6, 2, 1100, 64, theta=1e4, causal=False, backward=True, seed_id=428), lambda nb: bigbird_blocks(nb, seed=16), 3),
    (W("bsb_onepass_bigbird_causal_d128", 1, 8, 2, 1100, 128, theta=5e5, backward=True, seed_id=429), lambda nb: bigbird_blocks(nb, seed=17, causal=True), 3),
    (W("bsb_onepass_window_alibi", 1, 4, 2, 900, 128, theta=1e4, window=300, alibi=True, backward=True, seed_id=431), lambda nb: np.tril(np.ones((nb, nb), bool)), 3),
]


@pytest.mark.parametrize("w,pattern,tier", BWD_CASES, ids=lambda x: x.name if hasattr(x, "name") else "")
def test_block_sparse_backward(w, pattern, tier):
    run_bwd(w, pattern((w.S + 127) // 128), workspace_tier=tier)


def test_block_sparse_backward_empty_lists_give_zero_gradient_rows():
    w = W("bsb_empty", 1, 4, 2, 512, 128, theta=1e4, causal=False, backward=True, seed_id=430)
    a = np.zeros((4, 4), dtype=bool)
    a[0, 1] = a[2, 0] = a[2, 3] = True      # query blocks 1, 3 and key block 2 are never touched
    run_bwd(w, a)
    run_bwd(w, a, workspace_tier=3)


def test_bigbird_n4096_forward_and_backward():
    """The paper's block-sparse workload: a BigBird mask over 32 x 32 blocks at N = 4096 (about 8 % of the
    blocks active), RoPE on, full size in the launch configuration the bench times."""
    w = W("bigbird_4096", 1, 8, 2, 4096, 128, theta=5e5, causal=False, backward=True, seed_id=431)
    a = bigbird_blocks(32, window=1, n_global=0, n_random=0, seed=21)
    a[0, :] = True
    a[:, 0] = True      # one global block row and column; band of three: (3 * 32 - 2 + 62) / 1024 = 15 %
    run_bwd(w, a)
