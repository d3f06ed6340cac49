"""The allocation-free dispatch entry point against the plan-based one.

`moe_dispatch_tables_static` serves callers that cannot allocate device memory when they need
the tables (a decoding loop that must not hit cudaMalloc's device-wide synchronisation, or a
component with buffers and a stream but no allocator, which therefore cannot own a plan).  Its
scratch is one fixed array inside the library that all calls share and that keeps the previous
call's contents, so the test makes several calls in a row, smaller ones after larger ones.
What is expected comes from the CPU oracle's dispatch (the integer definition written out as
two loops), applied to indices the oracle selected; the plan-based entry point
`moe_route_from_logits` must give the same tables.  Integer tables: the comparison is bit-exact,
as in the other routing tests.  Collected last (file name) so an earlier failure cannot hide it.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import moe_oracle as orc
from paper_2509_02753_b200 import binding as B

pytestmark = pytest.mark.gpu


def _tables_from_plan(T, E, k, seed):
    """(idx on the device, counts, offsets, perm): expected tables from the oracle; the plan-based
    entry point is checked against them on the way."""
    g = torch.Generator().manual_seed(seed)
    logits = torch.randn((T, E), generator=g, dtype=torch.float32)
    idx_o, _, _ = orc.topk_gates(logits.numpy(), k, False, select_f32=True)
    counts_o, offsets_o, perm_o, _ = orc.dispatch(idx_o, E)
    with B.MoEPlan(64, E, 64, T, k, torch.float32) as plan:
        idx, _, counts, offsets, perm = plan.route_from_logits(logits.cuda(), k, False)
        assert plan.device_status() == 0
    assert np.array_equal(idx.cpu().numpy(), idx_o)
    assert np.array_equal(counts.cpu().numpy(), counts_o) and np.array_equal(perm.cpu().numpy(), perm_o)
    dev = lambda a: torch.from_numpy(a).cuda()
    return dev(idx_o), dev(counts_o), dev(offsets_o), dev(perm_o)


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


def test_static_scratch_dispatch_skips_entries_outside_the_expert_range_visibly():
    """An index outside 0..E-1 is left out of the tables: the counts then sum to fewer than T * k_l
    pairs, offsets[E] says how many were placed, and perm beyond that many entries is not written -
    which is how a caller notices.  The placed pairs are those of the oracle's dispatch with the bad
    pair removed."""
    T, E, k = 300, 16, 2
    g = torch.Generator().manual_seed(3)
    idx = torch.stack([torch.randperm(E, generator=g)[:k] for _ in range(T)]).to(torch.int32)
    idx[17, 1] = E                                   # one pair names an expert that does not exist
    keep = np.ones(T * k, dtype=bool)
    keep[17 * k + 1] = False
    flat = idx.numpy().reshape(-1)
    order = [p for e in range(E) for p in range(T * k) if keep[p] and flat[p] == e]   # the definition
    counts_e = np.bincount(flat[keep], minlength=E).astype(np.int32)
    c = torch.full((E,), -7, dtype=torch.int32, device="cuda")
    o = torch.full((E + 1,), -7, dtype=torch.int32, device="cuda")
    p = torch.full((T * k,), -7, dtype=torch.int32, device="cuda")
    B.moe_dispatch_tables_static(idx.cuda(), E, c, o, p)
    torch.cuda.synchronize()
    assert np.array_equal(c.cpu().numpy(), counts_e)
    assert int(o[E]) == T * k - 1
    assert p.cpu().numpy()[:T * k - 1].tolist() == order
    assert int(p[T * k - 1]) == -7                   # the tail is left as the caller had it
    # the next call with valid indices is not affected by what the bad one left in the shared array
    idx_ok, counts, offsets, perm = _tables_from_plan(300, 16, 2, 5)
    B.moe_dispatch_tables_static(idx_ok, E, c, o, p)
    torch.cuda.synchronize()
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
