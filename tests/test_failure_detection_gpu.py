"""Bounded waits: a wait that nothing satisfies expires, is reported through the plan's
status, and leaves the device usable.  No kernel faults, traps or hangs."""
import pytest
import torch

from paper_2509_26538_b200 import binding as hb

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_context_survives():
    plan = hb.Plan(16, 16, 64, 16, 2, 5)
    try:
        assert plan.status() == 0
        assert hb.lib().hilberta_selftest_timeout(plan._h, None) == 0
        assert plan.status() == hb.ERR_TIMEOUT      # reported once ...
        assert plan.status() == 0                   # ... and cleared
        # the same plan and device keep working
        q, k, v = (torch.randn((1, 2, plan.S, 128), device="cuda").bfloat16() for _ in range(3))
        out = torch.empty_like(q)
        plan.bind_like(q)
        plan.forward(q, k, v, out)
        assert plan.status() == 0
        assert torch.isfinite(out.float()).all()
    finally:
        plan.destroy()
    assert hb.lib().hilberta_selftest_timeout(None, None) == hb.ERR_INVALID
