"""The multi-rank path on CPU: two gloo ranks shard the tokens, route their shard (the oracle stands in for the
device kernels here: this test is about the sharding and the count reduction, not the arithmetic) and must
reproduce the single-rank result."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2609_36301_b200 import inputs
from paper_2609_36301_b200.sharding import allreduce_counts, expert_range, gather_shard_reports, token_range


def test_token_range_partitions_exactly():
    for T in (0, 1, 7, 128, 1000):
        for world in (1, 2, 3, 8):
            spans = [token_range(T, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == T
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    case = inputs.gaussian_case(101, 32, 8, 64, 4, 1, seed=17)
    lo, hi = token_range(case.T, rank, world)
    res = oracle.route(case.X[lo:hi], case.R1, case.R2, case.k, case.gate_mode, nthreads=1)
    counts = torch.from_numpy(res.counts.copy())
    allreduce_counts(counts)
    gathered = [None] * world
    dist.all_gather_object(gathered, (lo, hi, res.idx, res.gate))
    if rank == 0:
        ret["counts"] = counts.numpy()
        ret["parts"] = gathered
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_one_rank():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(2, port, ret), nprocs=2, join=True)
    case = inputs.gaussian_case(101, 32, 8, 64, 4, 1, seed=17)
    whole = oracle.route(case.X, case.R1, case.R2, case.k, case.gate_mode)
    assert np.array_equal(ret["counts"], whole.counts)
    idx = np.concatenate([p[2] for p in sorted(ret["parts"], key=lambda p: p[0])])
    gate = np.concatenate([p[3] for p in sorted(ret["parts"], key=lambda p: p[0])])
    assert np.array_equal(idx, whole.idx)
    np.testing.assert_array_equal(gate, whole.gate)


def test_expert_range_partitions_on_multiples_of_eight():
    for M in (8, 64, 96, 1000, 131072):
        for world in (1, 2, 3, 8):
            spans = [expert_range(M, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == M
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            assert all(a[0] % 8 == 0 for a in spans)


def _expert_worker(rank, world, port, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    case = inputs.gaussian_case(37, 32, 8, 72, 5, 1, seed=23)
    lo, hi = expert_range(case.M, rank, world)
    # the oracle stands in for the device router on this rank's expert slice
    res = oracle.route(case.X, case.R1, np.ascontiguousarray(case.R2[:, lo:hi]), case.k, 1, nthreads=1)
    idx, val, lse = gather_shard_reports(torch.from_numpy(res.idx), torch.from_numpy(res.topval), torch.from_numpy(res.lse))
    bases = [expert_range(case.M, r, world)[0] for r in range(world)]
    glob = idx.numpy() + np.asarray(bases, dtype=np.int32)[:, None, None]
    merged = oracle.merge(glob, val.numpy(), lse.numpy(), case.M, case.gate_mode)
    if rank == 1:                                   # every rank holds the merged result; report a non-zero one
        ret["merged"] = merged
    dist.barrier()
    dist.destroy_process_group()


def test_two_expert_shards_merge_to_the_unsharded_route():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_expert_worker, args=(2, port, ret), nprocs=2, join=True)
    case = inputs.gaussian_case(37, 32, 8, 72, 5, 1, seed=23)
    whole = oracle.route(case.X, case.R1, case.R2, case.k, case.gate_mode)
    m_idx, m_gate, m_val, m_lse, m_counts = ret["merged"]
    assert np.array_equal(m_idx, whole.idx)
    np.testing.assert_allclose(m_gate, whole.gate, rtol=1e-12)
    np.testing.assert_allclose(m_lse, whole.lse, rtol=1e-13)
    assert np.array_equal(m_counts, whole.counts)
