"""A bounded device-side wait that runs out must end in a status word, not in a hang.

Every wait of the prefill kernels on an mbarrier gives up after a limit, raises the CTA's abort
flag, and the kernel unwinds (status word set, tensor memory released).  No valid input makes
that happen, so the library carries a test-only entry point (csrc/gdn_test_hooks.h, not in the
public header) that runs the same wait and the same unwind on a barrier nobody arrives at, with
a short limit.  Nothing here faults, traps or waits without a limit.
"""
import ctypes
import time

import pytest

pytestmark = pytest.mark.gpu


def test_bounded_wait_runs_out_and_reports_through_the_status_word():
    import torch

    import paper_2607_16831_b200 as gdn

    L = gdn.lib()
    fn = L.gdn_test_bounded_wait
    fn.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_longlong, ctypes.c_void_p]
    fn.restype = ctypes.c_int

    # the status word is word 0 of an ordinary (here: minimal) workspace
    ws = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    elapsed = torch.zeros(1, dtype=torch.int64, device="cuda")
    torch.cuda.synchronize()
    assert gdn.gdn_last_device_status(ws) == 0

    t0 = time.perf_counter()
    rc = fn(ws.data_ptr(), elapsed.data_ptr(), 20000, None)
    assert rc == gdn.GDN_OK
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0
    assert wall < 0.25, "the kernel with a 20,000-cycle limit took %.3f s" % wall

    clocks = int(elapsed.item())
    assert clocks >= 20000, "the wait must have given up (it reports -1 when the barrier completed)"
    assert clocks < 2_000_000, "gave up after %d clocks: far beyond the limit it was given" % clocks
    assert gdn.gdn_last_device_status(ws) == 1      # kStatusTimeout, and the read clears it
    assert gdn.gdn_last_device_status(ws) == 0

    # the context is intact: tensor memory was released and ordinary work runs
    from gdn_inputs import config
    from paper_2607_16831_b200 import harness

    res = harness.run_prefill(config("prefill_tiny"))
    assert res["device_status"] == 0
    # argument errors of the hook itself
    assert fn(None, None, 20000, None) == 1
    assert fn(ws.data_ptr(), None, -5, None) == 2
