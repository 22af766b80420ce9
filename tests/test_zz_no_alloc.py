"""galv_dp_search_static: the search on the library's built-in scratch array.

Meant for callers that may not allocate device memory (a plugin inside a host
application that owns the device heap, a latency path where an allocation could
stall the device, a process whose pool is already full): they pass inputs and
outputs only.  The result must be what galv_dp_search gives with a
caller-provided workspace — here on two different batches back to back, since
every call reuses the same array and must clear what the last one left behind.

Collected last on purpose, so a failure here cannot hide other tests' results.
"""
import ctypes as C

import numpy as np
import pytest

from paper_2504_03662_b200 import inputs

pytestmark = pytest.mark.gpu


def _run_both(galv, w, flags):
    import torch
    from paper_2504_03662_b200 import binding as gb
    from paper_2504_03662_b200.search import SearchBuffers
    ref = SearchBuffers(galv, w, flags)
    ref.dp_search()
    ref.backtrack()
    want = ref.results()
    got = SearchBuffers(galv, w, flags)
    got.workspace = None                                  # nothing for the call to lean on
    call = lambda: galv.galv_dp_search_static(got.shape, got.L, got.time_q, got.mem_q, got.trans_q, got.C, got.A,
                                              got.C_last, got.status)
    call()                                                # the first call on a device loads the kernels' modules and
    torch.cuda.synchronize()                              # looks the array's address up: not part of the claim
    free_before = torch.cuda.mem_get_info()[0]            # the driver's count of free device bytes: any allocation,
    call()                                                # by whichever allocator, would lower it
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    got.backtrack()
    have = got.results()
    for k in ("opt_cost", "plan", "mem_used", "status"):
        assert (have[k] == want[k]).all(), k
    # tables of flagged instances are left untouched by both entry points (uninitialised memory): skip them
    valid = (want["status"] & ~1) == 0
    for i in range(w.B):
        if not valid[i]:
            continue
        Li = int(w.L[i])
        assert torch.equal(got.C_last[i], ref.C_last[i]), i
        for name in ("C", "A"):
            a, b = getattr(got, name), getattr(ref, name)
            if a is not None:
                assert torch.equal(a[i, :Li], b[i, :Li]), (name, i)
    return have


def test_static_workspace_matches_caller_workspace_twice():
    import torch
    from paper_2504_03662_b200 import binding as gb
    assert torch.cuda.is_available()
    galv = gb.Galv(0)
    try:
        # first call: ragged batch with one flagged instance, full table kept
        w1 = inputs.random_tables(90, 7, 9, 12, 300, ragged=True, mem_lo=1, mem_hi=70)
        w1.time_q[2, 0, 0] = -3
        r1 = _run_both(galv, w1, gb.STORE_C_FULL)
        assert r1["status"][2] == gb.STATUS_BAD_INPUT
        # second call straight after, other shape, argmin table and the rolling two-layer buffer
        w2 = inputs.random_tables(91, 3, 6, 24, 500, mem_lo=0, mem_hi=90)
        _run_both(galv, w2, gb.STORE_ARGMIN)
        # and the first shape again: nothing of the second call may linger
        r3 = _run_both(galv, w1, gb.STORE_C_FULL | gb.STORE_ARGMIN)
        assert (r3["opt_cost"] == r1["opt_cost"]).all()
    finally:
        galv.close()


def test_static_workspace_refuses_what_does_not_fit():
    import torch
    from paper_2504_03662_b200 import binding as gb
    galv = gb.Galv(0)
    try:
        # rolling mode needs 2*B*S*m_pitch*4 bytes of scratch: far beyond the built-in array here
        shape = gb.make_shape(64, 8, 32, 4095, gb.STORE_ARGMIN)
        assert galv.galv_dp_workspace_bytes(shape) > gb.STATIC_WORKSPACE_BYTES
        dummy = torch.zeros(64, dtype=torch.int32, device="cuda")
        rc = galv.lib.galv_dp_search_static(galv.h, C.byref(shape), *([dummy.data_ptr()] * 8), None)   # 8 arrays + the stream
        assert rc == gb.ERR_WORKSPACE
        assert b"GALV_STATIC_WORKSPACE_BYTES" in galv.lib.galv_last_error(galv.h)
        torch.cuda.synchronize()
    finally:
        galv.close()
