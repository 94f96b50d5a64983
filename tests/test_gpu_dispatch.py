"""Dispatch bookkeeping on the GPU (``more_dispatch``) against the oracle's stable counting sort.

Offsets are exact integers and must match bit for bit.  The order of pairs inside one expert's run is unspecified
on the GPU (atomic increments), so each run is compared as a set, and the whole list must be a permutation of the
valid pairs with non-decreasing expert ids."""
import numpy as np
import pytest

import oracle
from paper_2609_36301_b200 import binding as mr
from paper_2609_36301_b200 import inputs

from helpers import to_device

pytestmark = pytest.mark.gpu


def _check(idx_np, counts_np, offsets, pairs, M):
    ref_off, ref_pairs = oracle.dispatch(idx_np, M)
    assert np.array_equal(offsets.astype(np.int64), ref_off)
    n = int(ref_off[M])
    got = pairs[:n].astype(np.int64)
    flat = idx_np.ravel()
    assert np.array_equal(np.sort(got), np.sort(ref_pairs))                 # a permutation of the valid pairs
    assert np.all(np.diff(flat[got]) >= 0)                                  # grouped by expert
    # run by run: same members (sorting inside each run = sorting by (expert, position))
    assert np.array_equal(got[np.lexsort((got, flat[got]))], ref_pairs)
    assert np.array_equal(np.diff(ref_off), counts_np.astype(np.int64))


@pytest.mark.parametrize("T,h,r,M,k", [(256, 128, 8, 256, 2), (1000, 64, 16, 4096, 8), (3000, 64, 8, 40, 5), (1, 8, 8, 8, 1)])
def test_dispatch_after_routing(T, h, r, M, k):
    import torch
    case = inputs.gaussian_case(T, h, r, M, k, 0, seed=51)
    X, R1, R2 = to_device(case)
    res = mr.route(X, R1, R2, k, 0)
    offsets = torch.full((M + 1,), -1, dtype=torch.int32, device="cuda")
    pairs = torch.full((T * k,), -1, dtype=torch.int32, device="cuda")
    mr.more_dispatch(res.idx, res.counts, offsets, pairs)
    torch.cuda.synchronize()
    _check(res.idx.cpu().numpy(), res.counts.cpu().numpy(), offsets.cpu().numpy(), pairs.cpu().numpy(), M)


def test_dispatch_skewed_load_full_size():
    """The mixture workload (hot experts with thousands of pairs) at full size."""
    import torch
    case = inputs.make_config("c3", T=16384)
    X, R1, R2 = to_device(case)
    res = mr.route(X, R1, R2, case.k, 0)
    offsets = torch.empty((case.M + 1,), dtype=torch.int32, device="cuda")
    pairs = torch.empty((case.T * case.k,), dtype=torch.int32, device="cuda")
    for _ in range(2):                                                       # repeated calls reuse the cursor scratch
        mr.more_dispatch(res.idx, res.counts, offsets, pairs)
    torch.cuda.synchronize()
    _check(res.idx.cpu().numpy(), res.counts.cpu().numpy(), offsets.cpu().numpy(), pairs.cpu().numpy(), case.M)
    assert int(res.counts.max()) > 5 * case.T * case.k // case.M             # the load really is skewed


def test_dispatch_ignores_ids_outside_the_expert_range():
    import torch
    idx = torch.tensor([[0, 9], [2**31 - 1, 1], [1, -3]], dtype=torch.int32, device="cuda")
    counts = torch.tensor([1, 2, 0, 0], dtype=torch.int32, device="cuda")
    offsets = torch.empty((5,), dtype=torch.int32, device="cuda")
    pairs = torch.full((6,), -1, dtype=torch.int32, device="cuda")
    mr.more_dispatch(idx, counts, offsets, pairs)
    torch.cuda.synchronize()
    assert offsets.tolist() == [0, 1, 3, 3, 3]
    got = pairs.tolist()
    assert got[0] == 0 and sorted(got[1:3]) == [3, 4] and got[3:] == [-1, -1, -1]
