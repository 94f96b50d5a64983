"""Decode-sized batches and the expert-split merge at its widest: a handful of tokens, tens of thousands of experts,
the expert range cut over up to 64 CTAs per token block (plus the ranges swept side by side inside a CTA), the
partial top-k lists and (max, sum) pairs merged by the CTA that finishes last.  Every token is compared with the
oracle, including the log-sum-exp, with the automatic plan and with the split forced to its maximum."""
import numpy as np
import pytest

from paper_2609_36301_b200 import binding as mr
from paper_2609_36301_b200 import inputs

from helpers import check_counts, check_rows, to_device

pytestmark = pytest.mark.gpu

SHAPES = [(2048, 64, 16384, 8), (4096, 64, 131072, 16)]      # h, r, M, k


@pytest.mark.parametrize("h,r,M,k", SHAPES)
@pytest.mark.parametrize("T", [1, 64, 256])
@pytest.mark.parametrize("msplit", [0, 64])
@pytest.mark.parametrize("gate_mode", [0, 1])
def test_decode_shapes(T, h, r, M, k, msplit, gate_mode):
    import torch
    case = inputs.gaussian_case(T, h, r, M, k, gate_mode, seed=77)
    X, R1, R2 = to_device(case)
    plan = mr.more_route_plan_ex(T, h, r, M, k, gate_mode, True, mr.PATH_TCGEN05, msplit)
    if msplit == 0:
        assert plan.msplit * plan.expert_ranges >= 8, "a decode-sized batch must be spread along the expert axis"
    else:
        assert plan.msplit == 64
    res = mr.route(X, R1, R2, k, gate_mode, want_topval=True, want_lse=True, path=mr.PATH_TCGEN05, msplit=msplit)
    torch.cuda.synchronize()
    assert mr.more_route_status() == 0
    idx, gate, counts = res.idx.cpu().numpy(), res.gate.cpu().numpy(), res.counts.cpu().numpy()
    st = check_rows(case, None, idx, gate, res.topval.cpu().numpy(), res.lse.cpu().numpy(), gate_mode=gate_mode, k=k)
    check_counts(idx, counts, M, st["ref"].counts, any_differs=bool(st["differs_mask"].any()))
    # the same without the extra outputs (the variant without the softmax sweep in top-k mode)
    res2 = mr.route(X, R1, R2, k, gate_mode, path=mr.PATH_TCGEN05, msplit=msplit)
    torch.cuda.synchronize()
    assert mr.more_route_status() == 0
    assert np.array_equal(np.sort(res2.idx.cpu().numpy(), 1), np.sort(idx, 1))
    np.testing.assert_allclose(res2.gate.cpu().numpy(), gate, rtol=1e-4, atol=1e-7)
