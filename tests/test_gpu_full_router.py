"""The fused standard (full-rank) router on the GPU, ``more_route_full``, against the oracle.

The oracle has no separate standard router: with ``R1 = I_h`` (exact in bf16) its low-rank route IS the standard router
``softmax(TopK(X W))`` (the identity pin of the CPU tests), so the GPU result is checked against
``oracle.route(X, I, W)`` with the same acceptance rule as the low-rank path."""
import numpy as np
import pytest

from paper_2609_36301_b200 import binding as mr
from paper_2609_36301_b200 import inputs

from helpers import check_counts, check_rows, to_device

pytestmark = pytest.mark.gpu


def _run(case, msplit=0, gate_mode=None):
    import torch
    gm = case.gate_mode if gate_mode is None else gate_mode
    X, _, W = to_device(case)
    T, M, k = case.T, case.M, case.k
    idx = torch.full((T, k), -3, dtype=torch.int32, device="cuda")
    gate = torch.full((T, k), -1.0, dtype=torch.float32, device="cuda")
    counts = torch.full((M,), 77, dtype=torch.int32, device="cuda")
    topval = torch.empty((T, k), dtype=torch.float32, device="cuda")
    lse = torch.empty((T,), dtype=torch.float32, device="cuda")
    mr.more_route_full(X, W, k, gm, idx, gate, counts, topval, lse, msplit)
    torch.cuda.synchronize()
    assert mr.more_route_status() == 0
    stats = check_rows(case, None, idx.cpu().numpy(), gate.cpu().numpy(), topval.cpu().numpy(), lse.cpu().numpy(),
                       gate_mode=gm)
    check_counts(idx.cpu().numpy(), counts.cpu().numpy(), M, stats["ref"].counts, bool(stats["differs_mask"].any()))
    return stats


@pytest.mark.parametrize("gate_mode", [0, 1])
@pytest.mark.parametrize("T,h,M,k", [
    (256, 128, 256, 2),        # one CTA, one full 256-expert step, two k-tiles
    (300, 136, 200, 4),        # ragged everywhere: h not a multiple of 64, M not of 64, T not of 32
    (1000, 512, 1024, 8),      # several CTAs, eight k-tiles through three stages
    (2500, 64, 4096, 8),       # one k-tile per step
    (129, 256, 72, 16),        # list capacity 16, a token group with one live row
    (64, 384, 64, 32),         # list capacity 32, a single step
    (600, 192, 1000, 8),       # four 256-expert steps, the last one ragged (232 experts)
    (260, 128, 520, 4),        # three steps, eight live columns in the last; a second token group with four rows
])
def test_full_router_matches_oracle(T, h, M, k, gate_mode):
    case = inputs.full_rank_case(T, h, M, k, gate_mode, seed=5)
    stats = _run(case)
    assert stats["topval_err"] < 5e-5


@pytest.mark.parametrize("msplit", [2, 3, 7])
def test_full_router_with_expert_split(msplit):
    case = inputs.full_rank_case(700, 256, 2048, 8, 1, seed=9)
    _run(case, msplit=msplit)


def test_full_router_agrees_with_low_rank_router_on_the_identity():
    """Same inputs through ``more_route_ex`` with R1 = I (r = h = 64, the largest the low-rank tensor path takes):
    the two GPU paths must pick the same experts."""
    import torch
    case = inputs.full_rank_case(512, 64, 1024, 8, 0, seed=3)
    X, R1, W = to_device(case)
    low = mr.route(X, R1, W, case.k, 0)
    idx = torch.empty((case.T, case.k), dtype=torch.int32, device="cuda")
    gate = torch.empty((case.T, case.k), dtype=torch.float32, device="cuda")
    counts = torch.empty((case.M,), dtype=torch.int32, device="cuda")
    mr.more_route_full(X, W, case.k, 0, idx, gate, counts)
    torch.cuda.synchronize()
    same = (torch.sort(idx, dim=1).values == torch.sort(low.idx, dim=1).values).all(dim=1)
    assert same.float().mean() > 0.999                       # near-ties may differ; the oracle test is the exact one
    assert int(counts.sum()) == case.T * case.k


def test_full_router_rejects_shapes_it_cannot_take():
    import torch
    X = torch.zeros((8, 12), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((12, 16), dtype=torch.bfloat16, device="cuda")
    idx = torch.empty((8, 2), dtype=torch.int32, device="cuda")
    gate = torch.empty((8, 2), dtype=torch.float32, device="cuda")
    counts = torch.empty((16,), dtype=torch.int32, device="cuda")
    with pytest.raises(mr.MoreRouteError):
        mr.more_route_full(X, W, 2, 0, idx, gate, counts)     # h = 12 is not a multiple of 8


def test_full_router_at_benchmark_size_sampled_rows():
    """A full-size launch (c2's shape with M = 4096: 147 token blocks of 224 tokens, split in two along the experts, two
    CTAs per SM), checked on sampled rows the oracle can compute one by one and on the whole-output properties."""
    import torch
    T, h, M, k = 32768, 512, 4096, 8
    case = inputs.full_rank_case(T, h, M, k, 0, seed=21)
    X, _, W = to_device(case)
    idx = torch.empty((T, k), dtype=torch.int32, device="cuda")
    gate = torch.empty((T, k), dtype=torch.float32, device="cuda")
    counts = torch.empty((M,), dtype=torch.int32, device="cuda")
    topval = torch.empty((T, k), dtype=torch.float32, device="cuda")
    lse = torch.empty((T,), dtype=torch.float32, device="cuda")
    mr.more_route_full(X, W, k, 0, idx, gate, counts, topval, lse)
    torch.cuda.synchronize()
    assert mr.more_route_status() == 0
    rows = np.unique(np.concatenate([np.arange(0, 64), np.arange(T - 64, T),
                                     np.random.default_rng(4).integers(0, T, 128)]))
    idx_np, gate_np = idx.cpu().numpy(), gate.cpu().numpy()
    check_rows(case, rows, idx_np[rows], gate_np[rows], topval.cpu().numpy()[rows], lse.cpu().numpy()[rows], gate_mode=0)
    check_counts(idx_np, counts.cpu().numpy(), M)
    srt = np.sort(idx_np, axis=1)
    assert idx_np.min() >= 0 and idx_np.max() < M and np.all(srt[:, 1:] != srt[:, :-1])
    np.testing.assert_allclose(gate_np.sum(axis=1), 1.0, atol=1e-5)
