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
from paper_2609_36301_b200.sharding import allreduce_counts, token_range


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
