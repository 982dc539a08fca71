"""sage_select_static: selection for callers that cannot allocate device memory.

Some users of the library run where a device allocation at call time is not possible (all memory was
handed out at start-up by a pool they do not own, or none is left). For them the library offers a variant
of sage_select whose scratch is a fixed array inside the library. This test calls it through the C ABI and
checks it against sage_select on the same scores: the two are integer work on the same keys, so the indices
must be identical. It runs the pair twice in a row, with different scores and sizes, because every call
shares the one scratch array and must not depend on what the previous call left in it.

The file name sorts last on purpose: a run that stops at the first failure has then already run every
other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import paper_2510_02470_b200 as sage

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _scores(N, seed, ties):
    r = np.random.default_rng(seed)
    a = r.integers(-8, 9, N) / 8.0 if ties else r.uniform(-1.0, 1.0, N)
    return torch.from_numpy(a.astype(np.float32)).to(DEV)


def test_static_select_matches_allocating_select_twice_in_a_row():
    # two calls back to back on the shared scratch: a large tied case, then a smaller random one whose
    # keys and histogram occupy only part of what the first call wrote
    for N, rate, seed, ties in [(200000, 0.1, 1, True), (50001, 0.3, 2, False)]:
        s = _scores(N, seed, ties)
        k = sage.sage_select_count(N, rate)
        want = sage.sage_select(s, rate)
        got = sage.sage_select_static(s, rate, torch.empty((k,), dtype=torch.int64, device=DEV))
        torch.cuda.synchronize()
        assert got.numel() == k == want.numel()
        assert torch.equal(got, want), (N, rate)


def test_static_select_edges_and_limit():
    s = _scores(1000, 3, False)
    idx = torch.empty((1000,), dtype=torch.int64, device=DEV)
    for rate in (0.0, 1e-3, 1.0):
        assert torch.equal(sage.sage_select_static(s, rate, idx), sage.sage_select(s, rate))
    lib = sage.lib()
    k_out = C.c_int64(-7)
    big = 262144 + 1
    st = lib.sage_select_static(s.data_ptr(), big, 0.1, idx.data_ptr(), C.byref(k_out), None)
    assert st == 5 and k_out.value == -7                       # SAGE_ERR_UNSUPPORTED, out untouched
    assert b"262144" in lib.sage_last_error()
    assert lib.sage_select_static(None, 5, 0.5, idx.data_ptr(), None, None) == 1
    assert lib.sage_select_static(None, 0, 0.5, None, C.byref(k_out), None) == 0 and k_out.value == 0


def test_static_select_allocates_nothing_and_follows_the_stream():
    """What the entry point is for: after its first call on the device, further calls leave the device's free memory and
    torch's allocator untouched (the output buffer is the caller's, the scratch is inside the library), also when they
    are enqueued on a stream other than the default one."""
    s = _scores(100000, 5, False)
    k = sage.sage_select_count(100000, 0.25)
    idx = torch.empty((k,), dtype=torch.int64, device=DEV)
    want = sage.sage_select(s, 0.25)
    sage.sage_select_static(s, 0.25, idx)                        # first call on the device: looks up the array's address
    side = torch.cuda.Stream()                                   # the stream itself (torch's and the driver's doing) comes first
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        sage.sage_select_static(s, 0.25, idx)
    idx.zero_()
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    held0 = torch.cuda.memory_allocated()
    for i in range(4):
        idx.zero_()
        torch.cuda.synchronize()
        if i % 2:
            with torch.cuda.stream(side):
                got = sage.sage_select_static(s, 0.25, idx)
            side.synchronize()
        else:
            got = sage.sage_select_static(s, 0.25, idx)
            torch.cuda.synchronize()
        assert torch.equal(got, want)
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0 and torch.cuda.memory_allocated() == held0
