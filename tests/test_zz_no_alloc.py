"""The allocation-free dispatch entry point against the plan-based one.

`moe_dispatch_tables_static` serves callers that cannot allocate device memory when they need
the tables (a decoding loop that must not hit cudaMalloc's device-wide synchronisation, or a
component with buffers and a stream but no allocator, which therefore cannot own a plan).  Its
scratch is one fixed array inside the library that all calls share and that keeps the previous
call's contents, so the test makes two calls in a row, the second one smaller than the first,
and compares both with `moe_route_from_logits`.  Integer tables: the comparison is bit-exact,
as in the other routing tests.  Collected last (file name) so an earlier failure cannot hide it.
"""
import ctypes

import pytest
import torch

from paper_2509_02753_b200 import binding as B

pytestmark = pytest.mark.gpu


def _tables_from_plan(T, E, k, seed):
    g = torch.Generator().manual_seed(seed)
    logits = torch.randn((T, E), generator=g, dtype=torch.float32).cuda()
    with B.MoEPlan(64, E, 64, T, k, torch.float32) as plan:
        idx, _, counts, offsets, perm = plan.route_from_logits(logits, k, False)
        assert plan.device_status() == 0
    return idx, counts, offsets, perm


def test_static_scratch_dispatch_matches_plan_dispatch_twice_in_a_row():
    cases = [(4096, 60, 4, 11), (37, 8, 3, 12), (1, 128, 1, 13), (16384, 64, 4, 14)]
    expected = [_tables_from_plan(*c) for c in cases]
    # output buffers come from the caller; poison them so stale values cannot pass
    for (T, E, k, _), (idx, counts, offsets, perm) in zip(cases, expected):
        c = torch.full((E,), -7, dtype=torch.int32, device="cuda")
        o = torch.full((E + 1,), -7, dtype=torch.int32, device="cuda")
        p = torch.full((T * k,), -7, dtype=torch.int32, device="cuda")
        B.moe_dispatch_tables_static(idx, E, c, o, p)
        torch.cuda.synchronize()
        assert torch.equal(c, counts) and torch.equal(o, offsets) and torch.equal(p, perm)
        assert int(c.sum()) == T * k
    # and once more the first (largest-history) case, on a side stream
    T, E, k, _ = cases[0]
    idx, counts, offsets, perm = expected[0]
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    c = torch.zeros((E,), dtype=torch.int32, device="cuda")
    o = torch.zeros((E + 1,), dtype=torch.int32, device="cuda")
    p = torch.zeros((T * k,), dtype=torch.int32, device="cuda")
    with torch.cuda.stream(s):
        B.moe_dispatch_tables_static(idx, E, c, o, p, stream=s)
    s.synchronize()
    assert torch.equal(c, counts) and torch.equal(o, offsets) and torch.equal(p, perm)


def test_static_scratch_dispatch_rejects_sizes_beyond_its_array():
    lib = B.load_library()
    idx = torch.zeros((8, 2), dtype=torch.int32, device="cuda")
    buf = torch.zeros((70000 * 2,), dtype=torch.int32, device="cuda")
    call = lambda T, k, E: lib.moe_dispatch_tables_static(idx.data_ptr(), T, k, E, buf.data_ptr(),
                                                          buf.data_ptr(), buf.data_ptr(), None)
    assert call(65536 // 2 + 1, 2, 8) == -2        # T * k_l > 65536
    assert call(8, 2, 129) == -2                   # E > 128
    assert call(8, 0, 8) == -1 and call(8, 9, 8) == -1
    assert lib.moe_dispatch_tables_static(None, 8, 2, 8, buf.data_ptr(), buf.data_ptr(),
                                          buf.data_ptr(), None) == -1
