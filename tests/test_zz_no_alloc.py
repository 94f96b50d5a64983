"""The allocation-free entry point, checked against the ordinary one.

Some users of this library are not allowed to allocate device memory (their process budgets all of it through its
own pool, or a device allocation would stall their other streams), so ``more_route_noalloc`` keeps its scratch in a
fixed array inside the library.  That array is shared by all calls and is never cleared, which is exactly what could
go wrong: this test makes two calls in a row on different problems (the second smaller, so stale contents of the
first are still lying in the array) and requires each to agree with ``more_route_ex`` on the generic path, which runs
the same arithmetic out of ordinary scratch, and with the CPU oracle.  It lives in a file of its own that is collected last.
"""
import numpy as np
import pytest

from paper_2609_36301_b200 import binding as mr
from paper_2609_36301_b200 import inputs

from helpers import check_counts, check_rows

pytestmark = pytest.mark.gpu


def _dev(a):
    import torch
    return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)


def _run_both(case):
    import torch
    X, R1, R2 = _dev(case.X), _dev(case.R1), _dev(case.R2)
    k, gm = case.k, case.gate_mode
    ref = mr.route(X, R1, R2, k, gm, path=mr.PATH_GENERIC)
    idx = torch.full((case.T, k), -7, dtype=torch.int32, device="cuda")
    gate = torch.full((case.T, k), -7.0, dtype=torch.float32, device="cuda")
    counts = torch.full((case.M,), 12345, dtype=torch.int32, device="cuda")       # must be overwritten, not added to
    mr.more_route_noalloc(X, R1, R2, k, gm, idx, gate, counts)
    torch.cuda.synchronize()
    return ref, idx, gate, counts


def test_noalloc_matches_ordinary_entry_point_twice_in_a_row():
    import torch
    first = inputs.gaussian_case(1500, 192, 24, 1000, 8, 1, seed=41)     # T*r = 36000 floats of scratch
    second = inputs.gaussian_case(333, 72, 5, 130, 3, 0, seed=42)        # smaller: stale scratch beyond its reach
    for case in (first, second):
        ref, idx, gate, counts = _run_both(case)
        assert torch.equal(idx, ref.idx)
        assert torch.equal(counts, ref.counts)
        assert float((gate - ref.gate).abs().max()) <= 2e-3             # the tolerance of the parity tests
        assert int(counts.sum()) == case.T * case.k
        # ... and, in its own right, with the CPU oracle under the acceptance rule of the parity tests
        st = check_rows(case, None, idx.cpu().numpy(), gate.cpu().numpy(), gate_mode=case.gate_mode, k=case.k)
        check_counts(idx.cpu().numpy(), counts.cpu().numpy(), case.M, st["ref"].counts,
                     any_differs=bool(st["differs_mask"].any()))


def test_noalloc_rejects_problems_beyond_its_fixed_scratch():
    import torch
    cap = mr.more_route_noalloc_capacity()
    assert cap == 1 << 20
    T, r = 4097, 256                                                       # T*r just over the capacity
    X = torch.zeros((T, 64), dtype=torch.bfloat16, device="cuda")
    R1 = torch.zeros((64, r), dtype=torch.bfloat16, device="cuda")
    R2 = torch.zeros((r, 64), dtype=torch.bfloat16, device="cuda")
    idx = torch.empty((T, 2), dtype=torch.int32, device="cuda")
    gate = torch.empty((T, 2), dtype=torch.float32, device="cuda")
    counts = torch.full((64,), 9, dtype=torch.int32, device="cuda")
    with pytest.raises(mr.MoreRouteError) as err:
        mr.more_route_noalloc(X, R1, R2, 2, 0, idx, gate, counts)
    assert err.value.code == -8
    torch.cuda.synchronize()
    assert int(counts[0]) == 9                                             # nothing was touched
