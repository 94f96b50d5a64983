"""What stands in for a memory checker and a fault injector on a shared GPU: guard regions around every output (and
behind the library's own scratch) that must come back untouched, the bounded on-device wait made to run out on
purpose (by a wait that nothing can satisfy, not by a fault), and concurrent host threads on the staged entry point."""
import threading

import numpy as np
import pytest

from paper_2609_36301_b200 import binding as mr
from paper_2609_36301_b200 import inputs

from helpers import check_counts, check_rows, to_device

pytestmark = pytest.mark.gpu

GUARD = 1024          # elements of guard on either side of every output
PATTERN_I, PATTERN_F = -559038737, -12345.678


def guarded(torch, shape, dtype, pattern):
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * GUARD,), pattern, dtype=dtype, device="cuda")
    return buf, buf[GUARD:GUARD + n].view(*shape)


# ragged shapes, expert splits (inside and across CTAs), the largest k, more experts than the shared-memory histogram
# takes, both kernels of the low-rank router, the generic path
SHAPES = [
    # T,    h,   r,  M,     k,  msplit, path
    (129,   64,  8,  136,   2,  0, mr.PATH_TCGEN05),
    (515,   448, 56, 4104,  5,  3, mr.PATH_TCGEN05),
    (130,   128, 40, 776,   32, 0, mr.PATH_TCGEN05),
    (300,   256, 32, 65544, 8,  0, mr.PATH_TCGEN05),
    (64,    256, 64, 32768, 16, 64, mr.PATH_TCGEN05),
    (40000, 128, 16, 264,   8,  0, mr.PATH_TCGEN05),       # many tokens: the kernel with 256-token CTAs
    (70000, 64,  32, 2056,  8,  2, mr.PATH_TCGEN05),
    (33,    40,  8,  130,   5,  0, mr.PATH_GENERIC),
]


@pytest.mark.parametrize("T,h,r,M,k,msplit,path", SHAPES)
@pytest.mark.parametrize("gate_mode", [0, 1])
def test_nothing_is_written_outside_the_outputs(T, h, r, M, k, msplit, path, gate_mode):
    import torch
    case = inputs.gaussian_case(T, h, r, M, k, gate_mode, seed=13)
    X, R1, R2 = to_device(case)
    bi, idx = guarded(torch, (T, k), torch.int32, PATTERN_I)
    bg, gate = guarded(torch, (T, k), torch.float32, PATTERN_F)
    bc, counts = guarded(torch, (M,), torch.int32, PATTERN_I)
    bt, topval = guarded(torch, (T, k), torch.float32, PATTERN_F)
    bl, lse = guarded(torch, (T,), torch.float32, PATTERN_F)
    for with_extra in (True, False):
        mr.more_route_ex(X, R1, R2, k, gate_mode, idx, gate, counts, topval if with_extra else None,
                         lse if with_extra else None, path, msplit)
        torch.cuda.synchronize()
        assert mr.more_route_status() == 0
        for buf, pat in ((bi, PATTERN_I), (bg, PATTERN_F), (bc, PATTERN_I), (bt, PATTERN_F), (bl, PATTERN_F)):
            ref = torch.tensor(pat, dtype=buf.dtype, device="cuda")
            assert bool((buf[:GUARD] == ref).all()) and bool((buf[-GUARD:] == ref).all()), "guard region overwritten"
        assert mr.debug_scratch_guard() == 1, "the kernel wrote past the scratch bytes its plan asked for"
    # rows for the oracle: all of a small case, a sample of a large one
    rows = None if T <= 1000 else np.sort(np.random.default_rng(3).choice(T, size=512, replace=False))
    sel = slice(None) if rows is None else torch.from_numpy(rows).cuda()
    st = check_rows(case, rows, idx[sel].cpu().numpy(), gate[sel].cpu().numpy(), topval[sel].cpu().numpy(),
                    lse[sel].cpu().numpy(), gate_mode=gate_mode, k=k)
    check_counts(idx.cpu().numpy(), counts.cpu().numpy(), M)


def test_a_bounded_wait_that_runs_out_is_reported_once():
    """The time-out path of the kernels' mbarrier waits: a wait nobody can satisfy gives up after its budget, the
    kernel returns, more_route_status reports MORE_ERR_TIMEOUT exactly once and the library keeps working."""
    import torch
    assert mr.more_route_status() == 0
    assert mr.debug_expire_wait(200000) == 0          # ~0.1 ms of SM clocks
    torch.cuda.synchronize()                          # the kernel came back by itself
    assert mr.more_route_status() == -7
    assert mr.more_route_status() == 0                # reading the status clears it
    case = inputs.make_config("c0")
    X, R1, R2 = to_device(case)
    res = mr.route(X, R1, R2, case.k, 0, want_topval=True, want_lse=True)
    torch.cuda.synchronize()
    assert mr.more_route_status() == 0
    check_rows(case, None, res.idx.cpu().numpy(), res.gate.cpu().numpy(), res.topval.cpu().numpy(),
               res.lse.cpu().numpy(), gate_mode=0, k=case.k)


def test_host_entry_point_from_two_threads_with_different_sizes():
    """more_route_host shares one staging buffer per device; a call that grows it must not pull it from under a call
    that is still copying.  Two host threads, alternating a small and a large problem, every result checked."""
    import torch
    small = inputs.gaussian_case(300, 128, 16, 512, 4, 0, seed=5)
    large = inputs.gaussian_case(6000, 512, 32, 4096, 8, 1, seed=6)
    errors = []

    def worker(order):
        try:
            stream = torch.cuda.Stream()
            for case in order:
                idx = np.empty((case.T, case.k), dtype=np.int32)
                gate = np.empty((case.T, case.k), dtype=np.float32)
                counts = np.empty((case.M,), dtype=np.int32)
                mr.more_route_host(case.X, case.R1, case.R2, case.k, case.gate_mode, idx, gate, counts, stream)
                st = check_rows(case, None, idx, gate, gate_mode=case.gate_mode, k=case.k)
                check_counts(idx, counts, case.M, st["ref"].counts, any_differs=bool(st["differs_mask"].any()))
        except Exception as e:      # noqa: BLE001 - reported to the main thread
            errors.append(repr(e))

    torch.zeros(1, device="cuda")
    t1 = threading.Thread(target=worker, args=([small, large, small, large],))
    t2 = threading.Thread(target=worker, args=([large, small, large, small],))
    t1.start(); t2.start(); t1.join(); t2.join()
    assert not errors, errors
    assert mr.more_route_status() == 0


def test_a_call_that_fails_on_the_host_touches_no_output():
    """Every error the host can detect is detected before anything is enqueued: the outputs, out_counts included (which
    a successful call clears first), keep what they held.  Misaligned operand, a shape the forced tensor-core path
    cannot take, an expert split out of range, an unknown gate mode."""
    import torch
    T, h, r, M, k = 512, 256, 32, 1024, 8
    case = inputs.gaussian_case(T, h, r, M, k, 0, seed=5)
    X, R1, R2 = to_device(case)
    idx = torch.full((T, k), -3, dtype=torch.int32, device="cuda")
    gate = torch.full((T, k), -1.0, dtype=torch.float32, device="cuda")
    counts = torch.full((M,), 77, dtype=torch.int32, device="cuda")

    def untouched():
        torch.cuda.synchronize()
        return bool((idx == -3).all() and (gate == -1.0).all() and (counts == 77).all())

    # (1) X one bf16 element off a 16-byte boundary
    Xbig = torch.zeros((T * h + 8,), dtype=torch.bfloat16, device="cuda")
    Xoff = Xbig[1:1 + T * h].view(T, h)
    with pytest.raises(mr.MoreRouteError) as e:
        mr.more_route_ex(Xoff, R1, R2, k, 0, idx, gate, counts)
    assert e.value.code == -3 and untouched()          # MORE_ERR_ALIGN
    # (2) a rank the tensor-core path cannot take, with that path forced
    R1b = torch.zeros((h, 72), dtype=torch.bfloat16, device="cuda")
    R2b = torch.zeros((72, M), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mr.MoreRouteError) as e:
        mr.more_route_ex(X, R1b, R2b, k, 0, idx, gate, counts, path=mr.PATH_TCGEN05)
    assert e.value.code == -2 and untouched()          # MORE_ERR_SHAPE
    # (3) an expert split beyond the limit
    with pytest.raises(mr.MoreRouteError) as e:
        mr.more_route_ex(X, R1, R2, k, 0, idx, gate, counts, msplit=65)
    assert e.value.code == -2 and untouched()
    # (4) an unknown gate mode
    with pytest.raises(mr.MoreRouteError) as e:
        mr.more_route_ex(X, R1, R2, k, 7, idx, gate, counts)
    assert e.value.code == -4 and untouched()          # MORE_ERR_MODE
    # and the same buffers still work
    mr.more_route_ex(X, R1, R2, k, 0, idx, gate, counts)
    torch.cuda.synchronize()
    assert mr.more_route_status() == 0 and int(counts.sum()) == T * k
