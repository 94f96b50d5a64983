"""Small token counts on the grouped kernel: blocks of at most 64 tokens are repeated over the tensor-memory lanes (each
expert range of a CTA then works in another lane quarter), ranges shrink to a single 64-expert block, the first
buffers of a sweep are folded wholesale, and the partial lists of a token block are merged by the staged network
merge.  Token counts around the 32- and 64-token boundaries, every token against the oracle."""
import numpy as np
import pytest

from paper_2609_36301_b200 import binding as mr
from paper_2609_36301_b200 import inputs

from helpers import check_counts, check_rows, to_device

pytestmark = pytest.mark.gpu

SHAPES = [(128, 8, 256, 2), (256, 16, 1024, 4), (512, 32, 4096, 8), (320, 64, 2000, 8)]      # h, r, M, k


def _route_and_check(case, msplit):
    import torch
    X, R1, R2 = to_device(case)
    res = mr.route(X, R1, R2, case.k, case.gate_mode, want_topval=True, want_lse=True, path=mr.PATH_TCGEN05,
                   msplit=msplit)
    torch.cuda.synchronize()
    assert mr.more_route_status() == 0
    idx, gate, counts = res.idx.cpu().numpy(), res.gate.cpu().numpy(), res.counts.cpu().numpy()
    st = check_rows(case, None, idx, gate, res.topval.cpu().numpy(), res.lse.cpu().numpy(), gate_mode=case.gate_mode,
                    k=case.k)
    check_counts(idx, counts, case.M, st["ref"].counts, any_differs=bool(st["differs_mask"].any()))
    return st


@pytest.mark.parametrize("h,r,M,k", SHAPES)
@pytest.mark.parametrize("T", [1, 31, 33, 63, 65, 100, 130, 200])
@pytest.mark.parametrize("gate_mode", [0, 1])
def test_small_token_counts(T, h, r, M, k, gate_mode):
    case = inputs.gaussian_case(T, h, r, M, k, gate_mode, seed=1000 + T)
    plan = mr.more_route_plan_ex(T, h, r, M, k, gate_mode, True, mr.PATH_TCGEN05, 0)
    assert not plan.paired
    _route_and_check(case, 0)


@pytest.mark.parametrize("T", [1, 40, 64, 72, 100, 128, 250])
@pytest.mark.parametrize("msplit", [2, 8, 16])
def test_small_token_counts_with_forced_split(T, msplit):
    """Forced CTA splits of a 4096-expert sweep: 2 (serial merge), 8 and 16 (fanned-out network merge, 2 to 16 threads
    per token depending on the block size the plan picks)."""
    case = inputs.gaussian_case(T, 512, 32, 4096, 8, 1, seed=2000 + T + msplit)
    plan = mr.more_route_plan_ex(T, 512, 32, 4096, 8, 1, True, mr.PATH_TCGEN05, msplit)
    assert plan.msplit == msplit
    _route_and_check(case, msplit)


def test_equal_logits_across_expert_ranges_keep_the_lower_id():
    """Duplicated R2 columns in different expert ranges (and CTAs) give exactly equal logits: the merges must keep the
    lower id, as the oracle's total order does."""
    import torch
    T, h, r, M, k = 48, 256, 16, 2048, 4
    base = inputs.gaussian_case(T, h, r, M, k, 0, seed=31)
    R2 = base.R2.copy()
    R2[:, 1024:2048] = R2[:, 0:1024]            # expert j + 1024 is a copy of expert j
    case = inputs.RouterCase("duplicated-columns", base.X, base.R1, R2, k, 0, dict(base.meta))
    for msplit in (0, 4, 16):
        st = _route_and_check(case, msplit)
        assert not st["differs_mask"].any()


@pytest.mark.parametrize("T,h,r,M,k", [(1024, 1024, 32, 8192, 8), (512, 512, 32, 65536, 8), (1000, 256, 16, 16384, 4)])
@pytest.mark.parametrize("gate_mode", [0, 1])
def test_mid_sized_batches_split_over_many_ctas(T, h, r, M, k, gate_mode):
    """A few hundred to a thousand tokens with many experts: the plan splits every token block over 8 or more CTAs with
    64 to 128 tokens per block, so the last-arriver merge runs with two to four threads per token."""
    case = inputs.gaussian_case(T, h, r, M, k, gate_mode, seed=3000 + T)
    plan = mr.more_route_plan_ex(T, h, r, M, k, gate_mode, True, mr.PATH_TCGEN05, 0)
    assert not plan.paired and plan.msplit >= 8
    _route_and_check(case, 0)
