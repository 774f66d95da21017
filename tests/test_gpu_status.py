"""The time-out path of the boundary: a bounded device-side wait that runs out makes the kernel return, records a
code that the status calls report once, and leaves the context usable.  The wait is made to run out by a CTA
of the library's own self-test (a barrier that nothing arrives on, a limit of about a millisecond): nothing
here traps, faults or spins without a bound."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_13612_b200 as af
from paper_2609_13612_b200 import synth
import parity_util as pu

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_once_and_the_context_stays_usable():
    torch.cuda.synchronize()
    assert af.device_status()[0] == 0
    af.selftest_wait_timeout(2_000_000)          # about one millisecond of SM clocks
    code, detail = af.stream_status()            # in stream order behind the self-test launch
    assert code == 9, "expected AF_ERR_DEVICE_TIMEOUT, got %d" % code
    assert (detail >> 16) == 0x7e                # the wait site that gave up (not the warp released by the flag)
    assert (detail & 0xffff) == 0                # CTA 0
    assert af.stream_status() == (0, 0)          # cleared by the read
    assert af.device_status() == (0, 0)
    assert b"wait" in af.lib().attnfuse_strerror(9)
    # a normal forward afterwards is correct
    w = synth.Workload("after_timeout", 1, 4, 2, 300, 128, theta=1e4, seed_id=601)
    t = synth.draw_all(w)
    dev = {k: pu.to_dev(v) for k, v in t.items()}
    o, lse = pu.gpu_fwd(w, dev)
    want_o, want_l = oracle.run_workload(w, t)
    pu.assert_close("O after a timed-out wait", pu.to_np(o), want_o)
    assert np.abs(pu.to_np(lse) - want_l).max() <= pu.LSE_TOL


def test_device_status_reports_it_too():
    af.selftest_wait_timeout(1_000_000)
    code, detail = af.device_status()
    assert code == 9 and (detail >> 16) == 0x7e
    assert af.device_status() == (0, 0)


def test_selftest_rejects_unbounded_limits():
    for bad in (0, 10, 200_000_000):
        with pytest.raises(af.AttnFuseError) as e:
            af.selftest_wait_timeout(bad)
        assert e.value.code == 5
