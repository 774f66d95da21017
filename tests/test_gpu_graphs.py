"""The entry points can be captured into a CUDA graph (no allocation, no synchronisation inside the calls; the
programmatic dependent launches of the hybrid forward and of the backward sequence become graph edges) and a
replay reproduces the eager results bit for bit."""
import ctypes

import pytest
import torch

import paper_2609_13612_b200 as af
from paper_2609_13612_b200 import binding, synth
import parity_util as pu

pytestmark = pytest.mark.gpu
W = synth.Workload


def test_hybrid_forward_and_backward_in_a_cuda_graph():
    w = W("graph_fwd_bwd", 2, 8, 2, 640, 128, theta=5e5, backward=True, seed_id=151)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    sh = binding._Shape(w.B, w.Hq, w.Hkv, w.S, w.D)
    ws_f = torch.empty(af.lib().attnfuse_fwd_hybrid_workspace_bytes(ctypes.byref(sh)), dtype=torch.uint8, device="cuda")
    ws_b = torch.empty(af.lib().attnfuse_bwd_workspace_bytes(ctypes.byref(sh)), dtype=torch.uint8, device="cuda")
    o = torch.empty((w.B, w.Hq, w.S, w.D), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((w.B, w.Hq, w.S), dtype=torch.float32, device="cuda")

    def step():
        af.fwd_hybrid(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale, out=o, lse=lse, workspace=ws_f)
        return af.bwd(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale, workspace=ws_b)

    dq0, dk0, dv0 = step()
    torch.cuda.synchronize()
    o0, l0 = o.clone(), lse.clone()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            dq1, dk1, dv1 = step()
    o.zero_()
    lse.zero_()
    for x in (dq1, dk1, dv1):
        x.zero_()
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    assert torch.equal(o, o0) and torch.equal(lse, l0)
    assert torch.equal(dq1, dq0) and torch.equal(dk1, dk0) and torch.equal(dv1, dv0)


def test_one_pass_backward_in_a_cuda_graph():
    """The one-pass sequence (memset of the fp32 dQ accumulator, delta, two RoPE passes, the one-pass kernel, the finishing
    pass and the first-rows kernel, chained as programmatic dependents) captured and replayed: dK and dV bit-identical to
    the eager call, dQ up to the order of its fp32 reductions."""
    w = W("graph_onepass", 2, 8, 2, 640, 128, theta=5e5, backward=True, seed_id=152)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    rope, mask = pu.specs(w)
    table = af.rope_table(rope, w.S)
    ws = torch.empty(af.bwd_workspace_bytes(w.B, w.Hq, w.Hkv, w.S, w.D), dtype=torch.uint8, device="cuda")
    o, lse = af.fwd(dev["q"], dev["k"], dev["v"], rope, table, mask, w.scale)

    def step():
        with af.option(af.OPT_BWD_ONEPASS, 2):
            return af.bwd(dev["q"], dev["k"], dev["v"], o, lse, dev["do"], rope, table, mask, w.scale, workspace=ws)

    dq0, dk0, dv0 = step()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            dq1, dk1, dv1 = step()
    for x in (dq1, dk1, dv1):
        x.zero_()
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    assert torch.equal(dk1, dk0) and torch.equal(dv1, dv0)
    assert (dq1.float() - dq0.float()).abs().max().item() <= 2.0 ** -7 * dq0.float().abs().max().item()
