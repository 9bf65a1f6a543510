"""Failure detection without a GPU fault: device-side conditions land in the status word and the
context stays usable.  The bounded wait is made to run out on a barrier that nothing completes
(the library's own self-test kernel: one thread, nothing in flight)."""
import ctypes as C

import pytest
import torch

from paper_2302_00845_b200 import binding

pytestmark = pytest.mark.gpu


def test_bounded_wait_runs_out_and_reports_timeout():
    L = binding.lib()
    m, n, d = 4, 4, 4096
    with binding.CdGrab(m, n, d, "f32") as h:
        assert h.status() == binding.OK
        waited = C.c_longlong(0)
        limit = 2_000_000          # about a millisecond of SM clock
        assert L.cdgrab_selftest_wait_timeout(h._h, limit, C.byref(waited)) == binding.OK
        assert limit <= waited.value < 50 * limit         # gave up at the limit, not much later
        assert h.status() == binding.ERR_TIMEOUT          # sticky until cleared
        assert h.status() == binding.ERR_TIMEOUT
        # the context is still usable: a normal epoch runs and the flag can be cleared
        assert L.cdgrab_clear_status(h._h) == binding.OK
        assert h.status() == binding.OK
        h.begin_epoch()
        g = torch.randn(2, m, d, device="cuda")
        h.step(g); h.step(g)
        h.end_epoch()
        assert h.status() == binding.OK
        assert L.cdgrab_selftest_wait_timeout(h._h, 0, None) == binding.ERR_INVALID


def test_nonfinite_and_timeout_flags_are_independent():
    L = binding.lib()
    m, n, d = 2, 4, 4096
    with binding.CdGrab(m, n, d, "f32") as h:
        h.begin_epoch()
        g = torch.randn(2, m, d, device="cuda")
        g[1, 0, 5] = float("inf")
        h.step(g)
        assert h.status() == binding.ERR_NONFINITE
        assert L.cdgrab_selftest_wait_timeout(h._h, 100_000, None) == binding.OK
        assert h.status() == binding.ERR_TIMEOUT          # the time-out takes precedence in the report
        L.cdgrab_clear_status(h._h)
        assert h.status() == binding.OK
