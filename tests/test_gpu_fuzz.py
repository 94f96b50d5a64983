"""Seeded random shapes through the C interface against the oracle: the low-rank router on whichever path the plan
picks (tensor-core for h, r, M multiples of 8 and r <= 64, CUDA-core otherwise), forced expert splits, and the fused
standard router.  The shapes are drawn once from a fixed seed, so the cases are the same on every run."""
import numpy as np
import pytest

from paper_2609_36301_b200 import binding as mr
from paper_2609_36301_b200 import inputs

from helpers import check_counts, check_rows, to_device

pytestmark = pytest.mark.gpu


def _cases(n, seed, tensor_core):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        if tensor_core:
            h = int(rng.integers(1, 40)) * 8
            r = int(rng.choice([8, 16, 24, 32, 40, 48, 64]))
            M = int(rng.integers(1, 300)) * 8
        else:
            h = int(rng.integers(3, 200))
            r = int(rng.integers(1, 70))
            M = int(rng.integers(2, 1500))
        T = int(rng.integers(1, 700))
        k = int(min(M, rng.choice([1, 2, 3, 4, 6, 8, 8, 8, 12, 16, 20, 32])))
        gate_mode = int(rng.integers(0, 2))
        msplit = int(rng.choice([0, 0, 0, 1, 2, 3, 5]))
        out.append((T, h, r, M, k, gate_mode, msplit))
    return out


def _route_and_check(case, path, msplit):
    import torch
    X, R1, R2 = to_device(case)
    res = mr.route(X, R1, R2, case.k, case.gate_mode, want_topval=True, want_lse=True, path=path, msplit=msplit)
    torch.cuda.synchronize()
    assert mr.more_route_status() == 0
    idx = res.idx.cpu().numpy()
    stats = check_rows(case, None, idx, res.gate.cpu().numpy(), res.topval.cpu().numpy(), res.lse.cpu().numpy())
    check_counts(idx, res.counts.cpu().numpy(), case.M, stats["ref"].counts, bool(stats["differs_mask"].any()))


@pytest.mark.parametrize("T,h,r,M,k,gate_mode,msplit", _cases(24, 2024, True))
def test_random_shapes_tensor_core_path(T, h, r, M, k, gate_mode, msplit):
    case = inputs.gaussian_case(T, h, r, M, k, gate_mode, seed=T + M)
    plan = mr.more_route_plan(T, h, r, M, k, gate_mode, mr.PATH_TCGEN05, msplit)
    assert plan.path == mr.PATH_TCGEN05
    _route_and_check(case, mr.PATH_TCGEN05, msplit)


@pytest.mark.parametrize("T,h,r,M,k,gate_mode,msplit", _cases(12, 77, False))
def test_random_shapes_any_path(T, h, r, M, k, gate_mode, msplit):
    case = inputs.gaussian_case(T, h, r, M, k, gate_mode, seed=T + M)
    _route_and_check(case, mr.PATH_AUTO, 0)


@pytest.mark.parametrize("T,h,r,M,k,gate_mode,msplit", _cases(12, 4242, True))
def test_random_shapes_standard_router(T, h, r, M, k, gate_mode, msplit):
    import torch
    h = min(h, 256)                                         # the oracle forms z = X I_h: keep the identity small
    case = inputs.full_rank_case(T, h, M, k, gate_mode, seed=T + M)
    X, _, W = to_device(case)
    idx = torch.empty((T, k), dtype=torch.int32, device="cuda")
    gate = torch.empty((T, k), dtype=torch.float32, device="cuda")
    counts = torch.empty((M,), dtype=torch.int32, device="cuda")
    topval = torch.empty((T, k), dtype=torch.float32, device="cuda")
    lse = torch.empty((T,), dtype=torch.float32, device="cuda")
    mr.more_route_full(X, W, k, gate_mode, idx, gate, counts, topval, lse, msplit)
    torch.cuda.synchronize()
    assert mr.more_route_status() == 0
    stats = check_rows(case, None, idx.cpu().numpy(), gate.cpu().numpy(), topval.cpu().numpy(), lse.cpu().numpy())
    check_counts(idx.cpu().numpy(), counts.cpu().numpy(), M, stats["ref"].counts, bool(stats["differs_mask"].any()))
