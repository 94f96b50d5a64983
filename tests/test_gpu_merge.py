"""``more_merge_shards`` on the GPU: the global top-k of an expert-sharded router.

Two kinds of checks.  (1) The merge kernel alone against the oracle's merge on the same reports: ids and counts bit
for bit (the kernel compares the reported logits as they are), gates within the router's tolerance.  (2) The whole
sharded path through the C interface -- every shard routed by ``more_route_ex`` on its slice of R2, reports stacked,
merged -- against the unsharded oracle route, with the acceptance rule of the other parity tests."""
import numpy as np
import pytest

import oracle
from paper_2609_36301_b200 import binding as mr
from paper_2609_36301_b200 import inputs
from paper_2609_36301_b200.sharding import expert_range

from helpers import GATE_ATOL, LSE_ATOL, check_counts, check_rows, to_device

pytestmark = pytest.mark.gpu


def _merge_on_gpu(idx, val, lse, base, M, gate_mode, k):
    import torch
    S, T, _ = idx.shape
    d_idx = torch.from_numpy(idx).cuda()
    d_val = torch.from_numpy(val.astype(np.float32)).cuda()
    d_lse = None if lse is None else torch.from_numpy(lse.astype(np.float32)).cuda()
    out_idx = torch.full((T, k), -7, dtype=torch.int32, device="cuda")
    out_gate = torch.full((T, k), -1.0, dtype=torch.float32, device="cuda")
    out_val = torch.empty((T, k), dtype=torch.float32, device="cuda")
    out_lse = torch.empty((T,), dtype=torch.float32, device="cuda") if lse is not None else None
    counts = torch.full((M,), 99, dtype=torch.int32, device="cuda")
    mr.more_merge_shards(d_idx, d_val, d_lse, base, M, gate_mode, out_idx, out_gate, counts, out_val, out_lse)
    torch.cuda.synchronize()
    return (out_idx.cpu().numpy(), out_gate.cpu().numpy(), out_val.cpu().numpy(),
            None if out_lse is None else out_lse.cpu().numpy(), counts.cpu().numpy())


@pytest.mark.parametrize("gate_mode", [0, 1])
@pytest.mark.parametrize("S,T,k,M", [(2, 300, 8, 64), (5, 1000, 3, 1000), (64, 129, 16, 4096), (1, 33, 32, 40), (3, 1, 1, 3)])
def test_merge_kernel_matches_the_oracle_merge(S, T, k, M, gate_mode):
    rng = np.random.default_rng(S * 1000 + k)
    # synthetic reports: every shard owns a contiguous id range and reports min(k, size) distinct ids of it; logits are
    # fp32 values drawn from few distinct levels so that equal logits across shards exercise the tie rule
    bounds = np.linspace(0, M, S + 1).astype(np.int64)
    idx = np.full((S, T, k), -1, dtype=np.int32)
    val = np.full((S, T, k), -np.inf, dtype=np.float32)
    for s in range(S):
        size = int(bounds[s + 1] - bounds[s])
        ks = min(k, size)
        for t in range(T):
            idx[s, t, :ks] = rng.choice(size, ks, replace=False)
        val[s, :, :ks] = (rng.integers(-8, 9, size=(T, ks)) / 4.0).astype(np.float32)
    lse = (rng.standard_normal((S, T)) + 4.0).astype(np.float32)
    base = [int(b) for b in bounds[:-1]]
    glob = idx + np.where(idx >= 0, np.asarray(base, dtype=np.int32)[:, None, None], 0)
    r_idx, r_gate, r_val, r_lse, r_counts = oracle.merge(glob, val.astype(np.float64), lse.astype(np.float64), M, gate_mode)
    g_idx, g_gate, g_val, g_lse, g_counts = _merge_on_gpu(idx, val, lse, base, M, gate_mode, k)
    assert np.array_equal(g_idx, r_idx)
    assert np.array_equal(g_counts.astype(np.int64), r_counts)
    assert np.array_equal(g_val, r_val.astype(np.float32))
    assert np.abs(g_gate - r_gate).max() <= GATE_ATOL
    rel = np.abs(g_gate - r_gate) <= 1e-3 * r_gate + 1e-7
    assert rel.all()
    assert np.abs(g_lse - r_lse).max() <= LSE_ATOL


@pytest.mark.parametrize("gate_mode", [0, 1])
@pytest.mark.parametrize("world", [2, 3, 8])
def test_sharded_route_plus_merge_equals_the_unsharded_route(world, gate_mode):
    import torch
    T, h, r, M, k = 2000, 256, 32, 4096, 8
    case = inputs.gaussian_case(T, h, r, M, k, gate_mode, seed=77)
    X, R1, R2 = to_device(case)
    idx = torch.empty((world, T, k), dtype=torch.int32, device="cuda")
    val = torch.empty((world, T, k), dtype=torch.float32, device="cuda")
    lse = torch.empty((world, T), dtype=torch.float32, device="cuda")
    base = []
    for rank in range(world):
        lo, hi = expert_range(M, rank, world)
        base.append(lo)
        res = mr.route(X, R1, R2[:, lo:hi].contiguous(), k, gate_mode, want_topval=True, want_lse=True)
        idx[rank], val[rank], lse[rank] = res.idx, res.topval, res.lse
    out_idx = torch.empty((T, k), dtype=torch.int32, device="cuda")
    out_gate = torch.empty((T, k), dtype=torch.float32, device="cuda")
    out_val = torch.empty((T, k), dtype=torch.float32, device="cuda")
    out_lse = torch.empty((T,), dtype=torch.float32, device="cuda")
    counts = torch.empty((M,), dtype=torch.int32, device="cuda")
    mr.more_merge_shards(idx, val, lse, base, M, gate_mode, out_idx, out_gate, counts, out_val, out_lse)
    torch.cuda.synchronize()
    stats = check_rows(case, None, out_idx.cpu().numpy(), out_gate.cpu().numpy(), out_val.cpu().numpy(),
                       out_lse.cpu().numpy(), gate_mode=gate_mode)
    check_counts(out_idx.cpu().numpy(), counts.cpu().numpy(), M, stats["ref"].counts, bool(stats["differs_mask"].any()))


def test_merge_rejects_bad_arguments():
    import torch
    idx = torch.zeros((2, 4, 2), dtype=torch.int32, device="cuda")
    val = torch.zeros((2, 4, 2), dtype=torch.float32, device="cuda")
    out_idx = torch.empty((4, 2), dtype=torch.int32, device="cuda")
    out_gate = torch.empty((4, 2), dtype=torch.float32, device="cuda")
    counts = torch.empty((8,), dtype=torch.int32, device="cuda")
    with pytest.raises(mr.MoreRouteError):                       # full-softmax gates need the shards' lse
        mr.more_merge_shards(idx, val, None, None, 8, 1, out_idx, out_gate, counts)
    with pytest.raises(mr.MoreRouteError):
        mr.more_merge_shards(idx, val, None, None, 8, 5, out_idx, out_gate, counts)
    big = torch.zeros((65, 1, 1), dtype=torch.int32, device="cuda")
    with pytest.raises(mr.MoreRouteError):
        mr.more_merge_shards(big, big.float(), None, None, 8, 0, out_idx[:1, :1], out_gate[:1, :1], counts)
