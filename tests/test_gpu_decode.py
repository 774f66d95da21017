"""GPU parity of Flash Decoding (split-KV partials + log-sum-exp combine, GQA heads packed into one MMA
tile) against the fp64 oracle: the decode result is the last row of exact attention over the cache."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_13612_b200 as af
from paper_2609_13612_b200 import synth
import parity_util as pu

pytestmark = pytest.mark.gpu


def draw(B, Hq, Hkv, N, D, seed, sigma=1.0):
    """q [B,Hq,D] and the cache k, v [B,Hkv,N,D]: bf16-rounded fp32 values, the generator of the other tests."""
    rng = lambda tid: np.random.Generator(np.random.PCG64(np.random.SeedSequence([20260913, seed, tid])))
    q = synth.round_to_bf16(rng(0).standard_normal((B, Hq, D), dtype=np.float32) * sigma)
    k = synth.round_to_bf16(rng(1).standard_normal((B, Hkv, N, D), dtype=np.float32) * sigma)
    v = synth.round_to_bf16(rng(2).standard_normal((B, Hkv, N, D), dtype=np.float32) * sigma)
    return q, k, v


def oracle_decode(q, k, v, scale, window=-1, slopes=None):
    """Exact attention of a query at position N - 1: row N - 1 of the oracle's causal forward."""
    B, Hq, D = q.shape
    N = k.shape[2]
    qf = np.zeros((B, Hq, N, D), dtype=np.float32)
    qf[:, :, N - 1] = q
    o, l = oracle.fwd(qf, k, v, rotary_dim=0, causal=True, window=window, slopes=slopes, scale=scale, rows=[N - 1])
    return o[:, :, 0], l[:, :, 0]


def run(B, Hq, Hkv, N, D, seed, window=-1, alibi=False, n_splits=0, sigma=1.0, strided=False):
    q, k, v = draw(B, Hq, Hkv, N, D, seed, sigma)
    scale = 1.0 / np.sqrt(D)
    slopes = (2.0 ** (-8.0 * (np.arange(Hq) + 1) / Hq)).astype(np.float32) if alibi else None
    qd, kd, vd = pu.to_dev(q), pu.to_dev(k), pu.to_dev(v)
    if strided:   # a cache with room for more keys than are in use: rows of a larger allocation
        cap = N + 96
        kb = torch.zeros((B, Hkv, cap, D), dtype=torch.bfloat16, device="cuda")
        vb = torch.full((B, Hkv, cap, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        kb[:, :, :N] = kd
        vb[:, :, :N] = vd
        kd, vd = kb[:, :, :N], vb[:, :, :N]
    mask = af.MaskSpec(True, window, torch.from_numpy(slopes).cuda() if alibi else None)
    o, lse = af.decode(qd, kd, vd, mask, scale, n_splits=n_splits)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    want_o, want_l = oracle_decode(q, k, v, scale, window, slopes)
    pu.assert_close("decode O", pu.to_np(o), want_o)
    assert np.abs(pu.to_np(lse) - want_l).max() <= pu.LSE_TOL
    return o, lse


CASES = [
    # B, Hq, Hkv, N, D
    dict(B=1, Hq=4, Hkv=1, N=128, D=128, seed=301),                       # one tile per warp, one split
    dict(B=1, Hq=8, Hkv=2, N=1000, D=128, seed=302),                      # ragged tail, several splits
    dict(B=2, Hq=8, Hkv=8, N=515, D=64, seed=303),                        # MHA (g = 1), D = 64
    dict(B=1, Hq=16, Hkv=1, N=700, D=128, seed=304),                      # g = 16: every MMA row is a head
    dict(B=1, Hq=6, Hkv=2, N=333, D=128, seed=305),                       # g = 3 (rows replicated cyclically)
    dict(B=1, Hq=4, Hkv=2, N=1, D=128, seed=306),                         # a single cached key
    dict(B=1, Hq=4, Hkv=2, N=37, D=64, seed=307),                         # shorter than a tile
    dict(B=1, Hq=8, Hkv=2, N=2048, D=128, seed=308, window=300),          # sliding window: early tiles skipped
    dict(B=1, Hq=8, Hkv=2, N=900, D=128, seed=309, alibi=True),           # ALiBi
    dict(B=1, Hq=8, Hkv=2, N=1500, D=128, seed=310, window=257, alibi=True),
    dict(B=1, Hq=8, Hkv=2, N=640, D=128, seed=311, n_splits=1),           # no split at all
    dict(B=1, Hq=8, Hkv=2, N=640, D=128, seed=312, n_splits=5),           # the last split is empty
    dict(B=2, Hq=8, Hkv=2, N=777, D=128, seed=313, strided=True),         # rows of a larger cache allocation
]


@pytest.mark.parametrize("c", CASES, ids=lambda c: "B%d_Hq%d_Hkv%d_N%d_D%d_%d" % (c["B"], c["Hq"], c["Hkv"], c["N"], c["D"], c["seed"]))
def test_decode_small(c):
    run(**c)


def test_decode_is_deterministic_and_independent_of_the_split_count_up_to_rounding():
    q, k, v = draw(1, 8, 2, 3000, 128, 320)
    qd, kd, vd = pu.to_dev(q), pu.to_dev(k), pu.to_dev(v)
    mask = af.MaskSpec(True, -1, None)
    a, la = af.decode(qd, kd, vd, mask, 0.0884)
    b, lb = af.decode(qd, kd, vd, mask, 0.0884)
    assert torch.equal(a, b) and torch.equal(la, lb)
    c, lc = af.decode(qd, kd, vd, mask, 0.0884, n_splits=3)
    assert (a.float() - c.float()).abs().max().item() <= 4e-3
    assert (la - lc).abs().max().item() <= 1e-4


@pytest.mark.parametrize("name,Hq,Hkv,N", [("llama3_8b", 32, 8, 4096), ("llama3_70b", 64, 8, 32768),
                                            ("mistral_7b", 32, 8, 16384)])
def test_decode_paper_geometries(name, Hq, Hkv, N):
    """The three geometries of the paper's Flash Decoding table (query length 1, D = 128), full size, in
    the launch configuration the bench times."""
    run(1, Hq, Hkv, N, 128, seed=330 + Hq + N // 4096)


def test_decode_argument_errors():
    q, k, v = draw(1, 8, 2, 256, 128, 340)
    qd, kd, vd = pu.to_dev(q), pu.to_dev(k), pu.to_dev(v)
    mask = af.MaskSpec(True, -1, None)
    with pytest.raises(af.AttnFuseError) as e:
        af.decode(qd, kd, vd, mask, 0.1, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.code == 6
    with pytest.raises(af.AttnFuseError) as e:
        af.decode(qd, kd, vd, mask, -1.0)
    assert e.value.code == 5


def test_decode_reuses_one_cleared_workspace_over_many_calls():
    """The ticket counters at the head of the workspace are cleared once (decode_workspace) and every call leaves
    them at zero: repeated calls on the same workspace, with changing inputs, all match the oracle; the last CTA
    to finish differs from call to call, the bits of the result do not."""
    B, Hq, Hkv, N, D = 2, 8, 2, 1900, 128
    ws = af.decode_workspace(B, Hq, Hkv, N, D)
    mask = af.MaskSpec(True, -1, None)
    first = None
    for it in range(6):
        q, k, v = draw(B, Hq, Hkv, N, D, 350 + (it % 2))
        qd, kd, vd = pu.to_dev(q), pu.to_dev(k), pu.to_dev(v)
        o, lse = af.decode(qd, kd, vd, mask, D ** -0.5, workspace=ws)
        torch.cuda.synchronize()
        assert af.device_status()[0] == 0
        assert int(ws[:256].view(torch.int32).abs().sum().item()) == 0      # counters back at zero
        want_o, want_l = oracle_decode(q, k, v, D ** -0.5)
        pu.assert_close("decode call %d" % it, pu.to_np(o), want_o)
        assert np.abs(pu.to_np(lse) - want_l).max() <= pu.LSE_TOL
        if it == 0:
            first = (o.clone(), lse.clone())
        if it == 2:
            assert torch.equal(o, first[0]) and torch.equal(lse, first[1])
