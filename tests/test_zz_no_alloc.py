"""The workspace-free backward entry point.

Some users of this library call it from places where they may not ask CUDA (or torch) for memory:
inside another framework's enqueue hook, in a serving loop whose pool is frozen, while somebody
else holds the allocator.  `attnfuse_bwd_static` serves them with scratch that lives inside the
library.  This test calls it through the C-ABI twice in a row, with different problems so that the
second call finds the first one's leftovers in the shared scratch, and checks each result against
the ordinary entry point on the same inputs.  It needs nothing from the other tests.
"""
import pytest
import torch

import paper_2609_13612_b200 as af
from paper_2609_13612_b200 import binding, synth
import parity_util as pu

pytestmark = pytest.mark.gpu
W = synth.Workload


def _one_call(w):
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    o, lse = pu.gpu_fwd(w, dev)
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    # The static entry always takes the set-up that needs delta alone; the ordinary entry takes that same
    # set-up when its workspace has room for delta only (4 bytes per query row, rounded up to 256).
    delta_only = torch.empty((4 * w.B * w.Hq * w.S + 255) // 256 * 256, dtype=torch.uint8, device="cuda")
    same_tier = af.bwd(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale,
                       dq_dtype=torch.bfloat16, dkv_dtype=torch.float32, workspace=delta_only)
    full_ws = pu.gpu_bwd(w, dev, o, lse, dq_dtype=torch.bfloat16, dkv_dtype=torch.float32)
    # the caller owns the outputs; poison them so that an entry point that wrote nothing is caught
    dq = torch.full_like(same_tier[0], float("nan"))
    dk = torch.full_like(same_tier[1], float("nan"))
    dv = torch.full_like(same_tier[2], float("nan"))
    torch.cuda.synchronize()
    af.bwd_static(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale, dq, dk, dv)
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    for name, got, same, full in zip(("dQ", "dK", "dV"), (dq, dk, dv), same_tier, full_ws):
        # same kernels, same set-up, same inputs: the same bits
        assert torch.equal(got, same), "%s %s differs from attnfuse_bwd with a delta-only workspace" % (w.name, name)
        # and within the tolerance of the parity tests of the default (full-workspace) call
        pu.assert_close("%s %s static vs full workspace" % (w.name, name), pu.to_np(got), pu.to_np(full))


def test_static_backward_matches_workspace_backward_on_two_calls_in_a_row():
    _one_call(W("static_a", 2, 8, 2, 640, 128, theta=5e5, backward=True, seed_id=301))
    _one_call(W("static_b", 1, 4, 4, 333, 64, theta=1e4, window=100, alibi=True, backward=True, seed_id=302))


def test_static_backward_at_a_size_whose_caches_would_not_fit_the_scratch():
    """B*Hq*S = 2^18 rows with D = 128: delta is 1 MiB, the rotated-K cache alone would be 16 MiB."""
    _one_call(W("static_large", 2, 16, 4, 8192, 128, theta=5e5, backward=True, seed_id=303))


def test_static_backward_rejects_problems_beyond_its_scratch():
    rows = binding.BWD_STATIC_MAX_ROWS
    B, Hq, S, D = 1, 8, rows // 8 + 128, 64
    x = torch.empty((B, Hq, S, D), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((B, Hq, S), dtype=torch.float32, device="cuda")
    g32 = torch.zeros((B, Hq, S, D), dtype=torch.float32, device="cuda")
    with pytest.raises(af.AttnFuseError) as e:
        af.bwd_static(x, x, x, x, lse, x, af.RopeSpec(), None, af.MaskSpec(), 0.125, torch.empty_like(x), g32, g32.clone())
    assert e.value.code == 10
    assert b"AF_BWD_STATIC_MAX_ROWS" in af.lib().attnfuse_strerror(10)
