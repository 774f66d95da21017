"""Pins for the fp64 CPU oracle: closed forms, invariants, brute force, a library
special case and finite differences.  None of them re-uses the oracle's own formula;
each is chosen so that a plausible slip (dropped term, wrong sign or index, transposed
operand, wrong head mapping) fails at least one."""
import math

import numpy as np
import pytest
import torch

import oracle


def rnd(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


# ---------------------------------------------------------------- RoPE (Sections 2, 4.1)

def test_rope_preserves_row_norm():
    x = rnd((2, 3, 50, 32), 1)
    for R in (32, 16, 2):
        y = oracle.rope(x, 10000.0, R, pos_offset=7)
        assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-13, atol=0)


def test_rope_position_zero_is_identity_and_tail_passes_through():
    x = rnd((1, 1, 1, 16), 2)
    assert np.array_equal(oracle.rope(x, 500000.0, 16, pos_offset=0), x)
    x = rnd((1, 2, 9, 16), 3)
    y = oracle.rope(x, 10000.0, 8, pos_offset=3)
    assert np.array_equal(y[..., 8:], x[..., 8:])
    assert not np.allclose(y[..., :8], x[..., :8])


def test_rope_R2_is_textbook_plane_rotation():
    # R = 2: one pair, frequency theta^0 = 1, so position p rotates (x0, x1) by p radians.
    x = rnd((1, 1, 6, 2), 4)
    y = oracle.rope(x, 12345.0, 2, pos_offset=2)
    for s in range(6):
        p = 2 + s
        rot = np.array([[math.cos(p), -math.sin(p)], [math.sin(p), math.cos(p)]])
        assert np.allclose(y[0, 0, s], rot @ x[0, 0, s], atol=1e-14)


def test_rope_R4_pairs_are_half_swap_not_interleaved():
    # Hand case, theta = 100, R = 4, p = 1: frequencies 1 and 100^(-1/2) = 0.1.
    # Half-swap pairs (0,2) at angle 1 and (1,3) at angle 0.1.
    x = np.array([1.0, 0.0, 0.0, 0.0]).reshape(1, 1, 1, 4)
    y = oracle.rope(x, 100.0, 4, pos_offset=1)[0, 0, 0]
    assert np.allclose(y, [math.cos(1.0), 0.0, math.sin(1.0), 0.0], atol=1e-15)
    x = np.array([0.0, 0.0, 0.0, 1.0]).reshape(1, 1, 1, 4)
    y = oracle.rope(x, 100.0, 4, pos_offset=1)[0, 0, 0]
    assert np.allclose(y, [0.0, -math.sin(0.1), 0.0, math.cos(0.1)], atol=1e-15)
    # golden fixture holds the same hand case in text form
    import os
    g = np.loadtxt(os.path.join(os.path.dirname(__file__), "golden", "rope_r4_hand_case.txt"))
    xin, want = g[0], g[1]
    got = oracle.rope(xin.reshape(1, 1, 1, 4), 100.0, 4, pos_offset=1)[0, 0, 0]
    assert np.allclose(got, want, atol=5e-13)


def test_rope_dot_depends_only_on_relative_position():
    q = rnd((1, 1, 1, 32), 5)
    k = rnd((1, 1, 1, 32), 6)
    def dot(m, n):
        return float(np.sum(oracle.rope(q, 10000.0, 32, pos_offset=m) * oracle.rope(k, 10000.0, 32, pos_offset=n)))
    base = dot(5, 2)
    for t in (1, 17, 4000):
        assert abs(dot(5 + t, 2 + t) - base) < 1e-10
    assert abs(dot(6, 2) - base) > 1e-3


def test_rope_inverse_is_transpose():
    x = rnd((1, 2, 11, 16), 7)
    y = oracle.rope(x, 10000.0, 16, pos_offset=5)
    assert np.allclose(oracle.rope(y, 10000.0, 16, pos_offset=5, inverse=True), x, atol=1e-13)
    # <R x, z> == <x, R^T z>
    z = rnd(x.shape, 8)
    lhs = np.sum(y * z)
    rhs = np.sum(x * oracle.rope(z, 10000.0, 16, pos_offset=5, inverse=True))
    assert abs(lhs - rhs) < 1e-10


# ---------------------------------------------------------------- forward

def test_causal_row0_is_v0_and_L0_is_s00():
    q, k, v = rnd((2, 4, 9, 8), 10), rnd((2, 2, 9, 8), 11), rnd((2, 2, 9, 8), 12)
    o, lse = oracle.fwd(q, k, v, theta=10000.0, rotary_dim=8, pos_offset=3, scale=0.3)
    for h in range(4):
        assert np.allclose(o[:, h, 0], v[:, h // 2, 0], atol=1e-14)
    qr = oracle.rope(q, 10000.0, 8, 3)
    kr = oracle.rope(k, 10000.0, 8, 3)
    s00 = 0.3 * np.einsum("bhd,bhd->bh", qr[:, :, 0], np.repeat(kr, 2, axis=1)[:, :, 0])
    assert np.allclose(lse[:, :, 0], s00, atol=1e-13)


def test_output_invariant_to_position_offset():
    q, k, v = rnd((1, 2, 24, 16), 13), rnd((1, 2, 24, 16), 14), rnd((1, 2, 24, 16), 15)
    ref = oracle.fwd(q, k, v, theta=500000.0, rotary_dim=16, pos_offset=0)
    for p0 in (1000, 32768 - 24):
        got = oracle.fwd(q, k, v, theta=500000.0, rotary_dim=16, pos_offset=p0)
        assert np.allclose(got[0], ref[0], atol=1e-9) and np.allclose(got[1], ref[1], atol=1e-9)


def test_window_edge_cases():
    S = 12
    q, k, v = rnd((1, 2, S, 8), 16), rnd((1, 1, S, 8), 17), rnd((1, 1, S, 8), 18)
    ref = oracle.fwd(q, k, v, rotary_dim=8)
    full = oracle.fwd(q, k, v, rotary_dim=8, window=S - 1)
    assert np.array_equal(ref[0], full[0]) and np.array_equal(ref[1], full[1])
    less = oracle.fwd(q, k, v, rotary_dim=8, window=S - 2)  # drops exactly (S-1, 0)
    assert np.array_equal(less[0][:, :, :-1], ref[0][:, :, :-1])
    assert not np.allclose(less[0][:, :, -1], ref[0][:, :, -1])
    w0 = oracle.fwd(q, k, v, rotary_dim=8, window=0)
    assert np.allclose(w0[0], np.repeat(v, 2, axis=1), atol=1e-14)


def brute(q, k, v, theta, R, p0, causal, window, slopes, scale):
    """Explicit S x S matrix, naive exp / sum (no max shift), interleaved-free RoPE built
    from complex multiplication: an independent formulation."""
    B, Hq, S, D = q.shape
    g = Hq // k.shape[1]
    def rot(x):
        y = x.copy()
        half = R // 2
        if half == 0:
            return y
        pos = p0 + np.arange(S)
        freq = theta ** (-np.arange(half) * 2.0 / R)
        z = (x[..., :half] + 1j * x[..., half:R]) * np.exp(1j * pos[:, None] * freq[None, :])
        y[..., :half], y[..., half:R] = z.real, z.imag
        return y
    qr, kr = rot(q), rot(k)
    o = np.zeros_like(q)
    lse = np.zeros(q.shape[:3])
    for b in range(B):
        for h in range(Hq):
            sc = scale * qr[b, h] @ kr[b, h // g].T
            e = np.zeros((S, S))
            for i in range(S):
                for j in range(S):
                    if causal and j > i:
                        continue
                    if window >= 0 and abs(i - j) > window:
                        continue
                    s = sc[i, j] + (slopes[h] * (j - i) if slopes is not None else 0.0)
                    e[i, j] = math.exp(s)
            o[b, h] = (e / e.sum(1, keepdims=True)) @ v[b, h // g]
            lse[b, h] = np.log(e.sum(1))
    return o, lse


@pytest.mark.parametrize("causal,window,alibi,R", [
    (True, -1, False, 4), (True, 3, True, 4), (False, -1, False, 2), (False, 2, True, 4), (True, 1, False, 0),
])
def test_brute_force_tiny(causal, window, alibi, R):
    S, D, Hq, Hkv = 8, 4, 4, 2
    q, k, v = 0.7 * rnd((2, Hq, S, D), 20), 0.7 * rnd((2, Hkv, S, D), 21), rnd((2, Hkv, S, D), 22)
    slopes = np.array([0.5, 0.25, 0.125, 0.0625]) if alibi else None
    got = oracle.fwd(q, k, v, theta=50.0, rotary_dim=R, pos_offset=2, causal=causal, window=window,
                     slopes=slopes, scale=0.45)
    want = brute(q, k, v, 50.0, R, 2, causal, window, slopes, 0.45)
    assert np.allclose(got[0], want[0], atol=1e-12)
    assert np.allclose(got[1], want[1], atol=1e-12)


def test_zero_queries_closed_forms():
    S, D = 10, 4
    q = np.zeros((1, 2, S, D))
    k, v = rnd((1, 2, S, D), 23), rnd((1, 2, S, D), 24)
    o, lse = oracle.fwd(q, k, v, rotary_dim=4)
    for i in range(S):
        assert np.allclose(o[0, :, i], v[0, :, : i + 1].mean(1), atol=1e-14)
        assert np.allclose(lse[0, :, i], math.log(i + 1), atol=1e-14)
    W = 3
    o, _ = oracle.fwd(q, k, v, rotary_dim=4, window=W)
    for i in range(S):
        assert np.allclose(o[0, :, i], v[0, :, max(0, i - W): i + 1].mean(1), atol=1e-14)
    # ALiBi: weights proportional to exp(-m_h (i - j)); scale must not touch the bias.
    slopes = np.array([0.5, 0.125])
    o, lse = oracle.fwd(q, k, v, rotary_dim=4, slopes=slopes, scale=7.0)
    for h in range(2):
        for i in range(S):
            w = np.exp(-slopes[h] * (i - np.arange(i + 1)))
            assert np.allclose(o[0, h, i], (w[:, None] * v[0, h, : i + 1]).sum(0) / w.sum(), atol=1e-13)
            assert abs(lse[0, h, i] - math.log(w.sum())) < 1e-13


def test_no_rope_equals_library_sdpa_with_gqa():
    B, Hq, Hkv, S, D = 2, 6, 2, 33, 16
    q, k, v = rnd((B, Hq, S, D), 25), rnd((B, Hkv, S, D), 26), rnd((B, Hkv, S, D), 27)
    o, lse = oracle.fwd(q, k, v, rotary_dim=0, scale=0.2)
    tq, tk, tv = (torch.from_numpy(x) for x in (q, k, v))
    tk, tv = tk.repeat_interleave(3, dim=1), tv.repeat_interleave(3, dim=1)
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=0.2).numpy()
    assert np.allclose(o, want, atol=1e-12)
    o2, _ = oracle.fwd(q, k, v, rotary_dim=0, scale=0.2, causal=False)
    want2 = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=False, scale=0.2).numpy()
    assert np.allclose(o2, want2, atol=1e-12)


def test_constant_v_and_row_subset():
    B, Hq, Hkv, S, D = 1, 4, 2, 40, 8
    q, k = rnd((B, Hq, S, D), 28), rnd((B, Hkv, S, D), 29)
    v = np.broadcast_to(rnd((B, Hkv, 1, D), 30), (B, Hkv, S, D)).copy()
    o, _ = oracle.fwd(q, k, v, rotary_dim=8, window=9, slopes=np.array([.5, .25, .1, .05]))
    assert np.allclose(o, np.repeat(v, 2, axis=1), atol=1e-13)
    v = rnd((B, Hkv, S, D), 31)
    full = oracle.fwd(q, k, v, rotary_dim=8, pos_offset=5)
    rows = [0, 1, 17, 39]
    sub = oracle.fwd(q, k, v, rotary_dim=8, pos_offset=5, rows=rows)
    assert np.array_equal(sub[0], full[0][:, :, rows]) and np.array_equal(sub[1], full[1][:, :, rows])


# ---------------------------------------------------------------- backward (Section 4.4)

def torch_naive(q, k, v, theta, R, p0, causal, window, slopes, scale):
    """Naive autograd graph: rotate_half formulation, masked_fill, softmax, matmul."""
    B, Hq, S, D = q.shape
    g = Hq // k.shape[1]
    def rot(x):
        if R == 0:
            return x
        pos = torch.arange(p0, p0 + S, dtype=torch.float64)
        inv = theta ** (-torch.arange(0, R, 2, dtype=torch.float64) / R)
        ang = torch.outer(pos, inv)
        cos, sin = torch.cat([ang.cos(), ang.cos()], -1), torch.cat([ang.sin(), ang.sin()], -1)
        xr, xp = x[..., :R], x[..., R:]
        half = torch.cat([-xr[..., R // 2:], xr[..., : R // 2]], -1)
        return torch.cat([xr * cos + half * sin, xp], -1)
    qr, kr = rot(q), rot(k).repeat_interleave(g, dim=1)
    s = scale * qr @ kr.transpose(-1, -2)
    i = torch.arange(S)[:, None]
    j = torch.arange(S)[None, :]
    if slopes is not None:
        s = s + torch.as_tensor(slopes, dtype=torch.float64)[None, :, None, None] * (j - i)
    keep = torch.ones(S, S, dtype=torch.bool)
    if causal:
        keep &= j <= i
    if window >= 0:
        keep &= (i - j).abs() <= window
    s = s.masked_fill(~keep, float("-inf"))
    return torch.softmax(s, -1) @ v.repeat_interleave(g, dim=1)


@pytest.mark.parametrize("causal,window,alibi,R,S", [
    (True, -1, False, 16, 128), (True, 20, True, 16, 96), (False, 7, True, 8, 40), (True, -1, False, 0, 33),
])
def test_backward_matches_autograd_on_naive_graph(causal, window, alibi, R, S):
    B, Hq, Hkv, D = 2, 4, 2, 16
    q, k, v, do = (rnd((B, Hq, S, D), 40), rnd((B, Hkv, S, D), 41), rnd((B, Hkv, S, D), 42),
                   rnd((B, Hq, S, D), 43))
    slopes = np.array([0.5, 0.25, 0.125, 0.0625]) if alibi else None
    tq, tk, tv = (torch.from_numpy(x).requires_grad_(True) for x in (q, k, v))
    out = torch_naive(tq, tk, tv, 10000.0, R, 11, causal, window, slopes, 0.25)
    out.backward(torch.from_numpy(do))
    o, _ = oracle.fwd(q, k, v, theta=10000.0, rotary_dim=R, pos_offset=11, causal=causal, window=window,
                      slopes=slopes, scale=0.25)
    assert np.allclose(o, out.detach().numpy(), atol=1e-12)
    dq, dk, dv = oracle.bwd(q, k, v, do, theta=10000.0, rotary_dim=R, pos_offset=11, causal=causal,
                            window=window, slopes=slopes, scale=0.25)
    assert np.allclose(dq, tq.grad.numpy(), atol=1e-11)
    assert np.allclose(dk, tk.grad.numpy(), atol=1e-11)
    assert np.allclose(dv, tv.grad.numpy(), atol=1e-11)


@pytest.mark.parametrize("window,alibi", [(-1, False), (5, True)])
def test_backward_finite_differences(window, alibi):
    B, Hq, Hkv, S, D = 1, 4, 2, 12, 8
    q, k, v, do = (rnd((B, Hq, S, D), 50), rnd((B, Hkv, S, D), 51), rnd((B, Hkv, S, D), 52),
                   rnd((B, Hq, S, D), 53))
    slopes = np.array([0.5, 0.25, 0.125, 0.0625]) if alibi else None
    kw = dict(theta=10000.0, rotary_dim=8, pos_offset=4, causal=True, window=window, slopes=slopes, scale=0.35)
    dq, dk, dv = oracle.bwd(q, k, v, do, **kw)

    def loss(q_, k_, v_):
        return float(np.sum(oracle.fwd(q_, k_, v_, **kw)[0] * do))

    rng = np.random.default_rng(54)
    h = 1e-6
    for name, x, grad in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        for _ in range(12):
            idx = tuple(rng.integers(0, n) for n in x.shape)
            xp, xm = x.copy(), x.copy()
            xp[idx] += h
            xm[idx] -= h
            args_p = {"q": q, "k": k, "v": v}
            args_m = dict(args_p)
            args_p[name], args_m[name] = xp, xm
            fd = (loss(args_p["q"], args_p["k"], args_p["v"]) - loss(args_m["q"], args_m["k"], args_m["v"])) / (2 * h)
            assert abs(fd - grad[idx]) <= 1e-6 * max(1.0, abs(fd)), (name, idx, fd, grad[idx])


def test_backward_structural_properties():
    B, Hq, Hkv, S, D = 1, 4, 2, 20, 8
    q, k, v, do = (rnd((B, Hq, S, D), 60), rnd((B, Hkv, S, D), 61), rnd((B, Hkv, S, D), 62),
                   rnd((B, Hq, S, D), 63))
    kw = dict(theta=10000.0, rotary_dim=8, pos_offset=0)
    dq, dk, dv = oracle.bwd(q, k, v, np.zeros_like(do), **kw)
    assert not dq.any() and not dk.any() and not dv.any()
    dq, dk, dv = oracle.bwd(q, k, v, do, **kw)
    assert np.allclose(dq[:, :, 0], 0.0, atol=1e-15)  # causal row 0 sees one key: softmax is constant
    # key row 0 of dV collects dO_0 of every head of the group with weight 1, plus later rows
    # permuting query heads inside a group permutes dQ and leaves dK, dV unchanged
    perm = [1, 0, 3, 2]
    dq2, dk2, dv2 = oracle.bwd(q[:, perm], k, v, do[:, perm], **kw)
    assert np.allclose(dq2, dq[:, perm], atol=1e-13)
    assert np.allclose(dk2, dk, atol=1e-12) and np.allclose(dv2, dv, atol=1e-12)
    # moving a query head to another group does change dK
    perm = [2, 1, 0, 3]
    _, dk3, _ = oracle.bwd(q[:, perm], k, v, do[:, perm], **kw)
    assert not np.allclose(dk3, dk, atol=1e-6)


# ---------------------------------------------------------------- block-sparse attention (Section 4.3)

def test_blocks_all_active_is_the_dense_result():
    q, k, v, do = rnd((1, 4, 24, 8), 60), rnd((1, 2, 24, 8), 61), rnd((1, 2, 24, 8), 62), rnd((1, 4, 24, 8), 63)
    kw = dict(theta=100.0, rotary_dim=8, pos_offset=3, causal=True, window=9, scale=0.3)
    ones = np.ones((6, 6))
    a, b = oracle.fwd(q, k, v, **kw), oracle.fwd(q, k, v, blocks=ones, block_size=4, **kw)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    ga, gb = oracle.bwd(q, k, v, do, **kw), oracle.bwd(q, k, v, do, blocks=ones, block_size=4, **kw)
    assert all(np.array_equal(x, y) for x, y in zip(ga, gb))


def test_block_diagonal_mask_is_independent_attention_per_block():
    """With only the diagonal blocks active (no causal rule) every block attends to itself: the same as
    running each block alone, at its own position offset (a ragged last block included)."""
    S, bs, D = 22, 8, 8
    q, k, v, do = rnd((1, 2, S, D), 64), rnd((1, 2, S, D), 65), rnd((1, 2, S, D), 66), rnd((1, 2, S, D), 67)
    nb = 3
    kw = dict(theta=50.0, rotary_dim=4, causal=False, scale=0.4)
    o, l = oracle.fwd(q, k, v, pos_offset=5, blocks=np.eye(nb), block_size=bs, **kw)
    dq, dk, dv = oracle.bwd(q, k, v, do, pos_offset=5, blocks=np.eye(nb), block_size=bs, **kw)
    for b0 in range(0, S, bs):
        sl = slice(b0, min(S, b0 + bs))
        ob, lb = oracle.fwd(q[:, :, sl], k[:, :, sl], v[:, :, sl], pos_offset=5 + b0, **kw)
        assert np.allclose(o[:, :, sl], ob, atol=1e-13) and np.allclose(l[:, :, sl], lb, atol=1e-13)
        gq, gk, gv = oracle.bwd(q[:, :, sl], k[:, :, sl], v[:, :, sl], do[:, :, sl], pos_offset=5 + b0, **kw)
        assert np.allclose(dq[:, :, sl], gq, atol=1e-13) and np.allclose(dk[:, :, sl], gk, atol=1e-13)
        assert np.allclose(dv[:, :, sl], gv, atol=1e-13)


def test_blocks_brute_force_and_autograd_tiny():
    """Random block pattern on top of the causal rule against an explicit masked softmax in torch
    (forward) and its autograd (backward); one query block has no active block at all."""
    S, bs, D, Hq, Hkv = 12, 3, 4, 4, 2
    q, k, v, do = rnd((2, Hq, S, D), 70), rnd((2, Hkv, S, D), 71), rnd((2, Hkv, S, D), 72), rnd((2, Hq, S, D), 73)
    blocks = np.array([[1, 0, 0, 0], [0, 0, 0, 0], [1, 0, 1, 0], [0, 1, 1, 1]])
    keep = np.kron(blocks, np.ones((bs, bs))).astype(bool) & (np.arange(S)[None, :] <= np.arange(S)[:, None])
    tq, tk, tv = (torch.from_numpy(x).requires_grad_(True) for x in (q, k, v))
    s = 0.5 * tq @ tk.repeat_interleave(2, dim=1).transpose(-1, -2)
    s = s.masked_fill(~torch.from_numpy(keep), float("-inf"))
    p = torch.nan_to_num(torch.softmax(s, -1), nan=0.0)      # rows without a kept pair: all zero
    out = p @ tv.repeat_interleave(2, dim=1)
    out.backward(torch.from_numpy(do))
    o, l = oracle.fwd(q, k, v, rotary_dim=0, causal=True, scale=0.5, blocks=blocks, block_size=bs)
    assert np.allclose(o, out.detach().numpy(), atol=1e-12)
    assert np.all(o[:, :, 3:6] == 0.0) and np.all(np.isneginf(l[:, :, 3:6]))
    dq, dk, dv = oracle.bwd(q, k, v, do, rotary_dim=0, causal=True, scale=0.5, blocks=blocks, block_size=bs)
    assert np.allclose(dq, tq.grad.numpy(), atol=1e-11) and np.allclose(dk, tk.grad.numpy(), atol=1e-11)
    assert np.allclose(dv, tv.grad.numpy(), atol=1e-11)
    assert np.all(dq[:, :, 3:6] == 0.0)


# ---------------------------------------------------------------- additive_bias, relu_attention, full (Section 3.1)

def _naive(q, k, v, keep, bias, scale, relu):
    """Explicit torch graph in fp64: scores, bias, mask, normaliser, P V (GQA by repeat_interleave)."""
    g = q.shape[1] // k.shape[1]
    s = scale * q @ k.repeat_interleave(g, dim=1).transpose(-1, -2)
    if bias is not None:
        s = s + bias
    if relu:
        n = keep.sum(-1, keepdim=True).clamp(min=1)
        p = torch.where(keep, torch.relu(s), torch.zeros_like(s)) / n
    else:
        p = torch.nan_to_num(torch.softmax(s.masked_fill(~keep, float("-inf")), -1), nan=0.0)
    return p @ v.repeat_interleave(g, dim=1)


def test_bias_filled_with_the_alibi_term_is_alibi():
    """additive_bias carrying slope_h * (j - i) gives what the ALiBi combinator gives, forward and backward."""
    S, D = 20, 8
    q, k, v, do = rnd((2, 4, S, D), 80), rnd((2, 2, S, D), 81), rnd((2, 2, S, D), 82), rnd((2, 4, S, D), 83)
    slopes = np.array([0.5, 0.25, 0.125, 0.0625])
    ji = (np.arange(S)[None, :] - np.arange(S)[:, None]).astype(np.float64)
    bias = slopes[None, :, None, None] * ji[None, None]
    kw = dict(theta=100.0, rotary_dim=8, pos_offset=2, causal=True, window=11, scale=0.3)
    a, b = oracle.fwd(q, k, v, slopes=slopes, **kw), oracle.fwd(q, k, v, bias=bias, **kw)
    assert np.allclose(a[0], b[0], atol=1e-13) and np.allclose(a[1], b[1], atol=1e-13)
    ga, gb = oracle.bwd(q, k, v, do, slopes=slopes, **kw), oracle.bwd(q, k, v, do, bias=bias, **kw)
    assert all(np.allclose(x, y, atol=1e-12) for x, y in zip(ga, gb))
    # a sign or transposition slip in the bias index would show: the transposed bias is a different result
    c = oracle.fwd(q, k, v, bias=np.swapaxes(bias, 2, 3), **kw)
    assert not np.allclose(a[0], c[0], atol=1e-6)


def test_bias_of_minus_infinity_is_a_mask_and_broadcasts():
    S, D = 14, 4
    q, k, v, do = rnd((2, 2, S, D), 84), rnd((2, 2, S, D), 85), rnd((2, 2, S, D), 86), rnd((2, 2, S, D), 87)
    causal_bias = np.where(np.arange(S)[None, :] <= np.arange(S)[:, None], 0.0, -np.inf)[None, None]
    kw = dict(rotary_dim=4, theta=50.0, scale=0.5)
    a = oracle.fwd(q, k, v, causal=True, **kw)
    b = oracle.fwd(q, k, v, causal=False, bias=causal_bias, **kw)                      # [1, 1, S, S] broadcast
    c = oracle.fwd(q, k, v, causal=False, bias=np.broadcast_to(causal_bias, (2, 2, S, S)).copy(), **kw)
    assert np.allclose(a[0], b[0], atol=1e-13) and np.allclose(a[1], b[1], atol=1e-13)
    assert np.array_equal(b[0], c[0]) and np.array_equal(b[1], c[1])
    ga = oracle.bwd(q, k, v, do, causal=True, **kw)
    gb = oracle.bwd(q, k, v, do, causal=False, bias=causal_bias, **kw)
    assert all(np.allclose(x, y, atol=1e-12) for x, y in zip(ga, gb))
    # `full` (no mask at all) is causal=False without a window: every pair kept
    full = oracle.fwd(q, k, v, causal=False, window=-1, **kw)
    assert not np.allclose(full[0], a[0], atol=1e-6)


def test_bias_per_batch_and_head_against_autograd():
    S, D, Hq, Hkv = 11, 4, 4, 2
    q, k, v, do = rnd((2, Hq, S, D), 88), rnd((2, Hkv, S, D), 89), rnd((2, Hkv, S, D), 90), rnd((2, Hq, S, D), 91)
    bias = rnd((2, Hq, S, S), 92)
    keep = torch.from_numpy(np.arange(S)[None, :] <= np.arange(S)[:, None])
    tq, tk, tv = (torch.from_numpy(x).requires_grad_(True) for x in (q, k, v))
    out = _naive(tq, tk, tv, keep, torch.from_numpy(bias), 0.7, relu=False)
    out.backward(torch.from_numpy(do))
    o, _ = oracle.fwd(q, k, v, rotary_dim=0, causal=True, scale=0.7, bias=bias)
    assert np.allclose(o, out.detach().numpy(), atol=1e-12)
    dq, dk, dv = oracle.bwd(q, k, v, do, rotary_dim=0, causal=True, scale=0.7, bias=bias)
    assert np.allclose(dq, tq.grad.numpy(), atol=1e-11) and np.allclose(dk, tk.grad.numpy(), atol=1e-11)
    assert np.allclose(dv, tv.grad.numpy(), atol=1e-11)
    # the head extent of the bias follows the QUERY head: permuting heads of q and bias together permutes O
    perm = [1, 0, 3, 2]
    o2, _ = oracle.fwd(q[:, perm], k, v, rotary_dim=0, causal=True, scale=0.7, bias=bias[:, perm])
    assert np.allclose(o2, o[:, perm], atol=1e-13)


def test_relu_attention_closed_forms_fix_the_normalisation():
    """With Q = 0 every score equals its bias.  A constant bias c > 0 gives O_i = c * mean of the kept values
    (relu(c) / n_i each): with the row's kept count n_i, not the sequence length, under a mask.  A negative
    constant gives O = 0."""
    S, D = 9, 3
    k, v = rnd((1, 1, S, D), 93), rnd((1, 1, S, D), 94)
    q = np.zeros((1, 2, S, D))
    c = 1.75
    o, l = oracle.fwd(q, k, v, rotary_dim=0, causal=True, scale=1.0, bias=np.full((1, 1, S, S), c), normaliser="relu")
    assert l is None
    for i in range(S):
        assert np.allclose(o[0, :, i], c * v[0, 0, :i + 1].mean(0), atol=1e-13)
    o, _ = oracle.fwd(q, k, v, rotary_dim=0, causal=True, window=2, scale=1.0, bias=np.full((1, 1, S, S), c), normaliser="relu")
    for i in range(S):
        assert np.allclose(o[0, :, i], c * v[0, 0, max(0, i - 2):i + 1].mean(0), atol=1e-13)
    o, _ = oracle.fwd(q, k, v, rotary_dim=0, causal=False, scale=1.0, bias=np.full((1, 1, S, S), c), normaliser="relu")
    assert np.allclose(o[0, 0], np.broadcast_to(c * v[0, 0].mean(0), (S, D)), atol=1e-13)   # full: n_i = S
    o, _ = oracle.fwd(q, k, v, rotary_dim=0, causal=True, scale=1.0, bias=np.full((1, 1, S, S), -c), normaliser="relu")
    assert not o.any()


def test_relu_attention_against_autograd_and_finite_differences():
    S, D, Hq, Hkv = 10, 4, 4, 2
    q, k, v, do = rnd((2, Hq, S, D), 95), rnd((2, Hkv, S, D), 96), rnd((2, Hkv, S, D), 97), rnd((2, Hq, S, D), 98)
    bias = 0.3 * rnd((1, Hq, S, S), 99)
    keep_np = (np.arange(S)[None, :] <= np.arange(S)[:, None]) & (np.arange(S)[:, None] - np.arange(S)[None, :] <= 6)
    tq, tk, tv = (torch.from_numpy(x).requires_grad_(True) for x in (q, k, v))
    out = _naive(tq, tk, tv, torch.from_numpy(keep_np), torch.from_numpy(bias), 0.6, relu=True)
    out.backward(torch.from_numpy(do))
    kw = dict(rotary_dim=0, causal=True, window=6, scale=0.6, bias=bias, normaliser="relu")
    o, _ = oracle.fwd(q, k, v, **kw)
    assert np.allclose(o, out.detach().numpy(), atol=1e-12)
    dq, dk, dv = oracle.bwd(q, k, v, do, **kw)
    assert np.allclose(dq, tq.grad.numpy(), atol=1e-11) and np.allclose(dk, tk.grad.numpy(), atol=1e-11)
    assert np.allclose(dv, tv.grad.numpy(), atol=1e-11)
    # with RoPE in front: central differences of sum(O * dO) (the kinks of relu have measure zero)
    kw = dict(theta=30.0, rotary_dim=4, pos_offset=1, causal=True, scale=0.6, normaliser="relu")
    dq, dk, dv = oracle.bwd(q, k, v, do, **kw)
    f = lambda a, b, c: float((oracle.fwd(a, b, c, **kw)[0] * do).sum())
    h = 1e-6
    r = np.random.default_rng(5)
    for (name, x, gx) in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        for _ in range(6):
            idx = tuple(r.integers(0, n) for n in x.shape)
            xp, xm = x.copy(), x.copy()
            xp[idx] += h
            xm[idx] -= h
            args_p = {"q": (xp, k, v), "k": (q, xp, v), "v": (q, k, xp)}[name]
            args_m = {"q": (xm, k, v), "k": (q, xm, v), "v": (q, k, xm)}[name]
            num = (f(*args_p) - f(*args_m)) / (2 * h)
            assert abs(num - gx[idx]) <= 1e-6 * max(1.0, abs(num)), (name, idx, num, gx[idx])
