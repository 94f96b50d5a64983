"""Algorithm 2's statistic psum = column sums of the softmax over all experts, on the GPU against the oracle.

psum is accumulated with floating-point atomics, so it is compared with a tolerance: relative 2e-4 plus a small
absolute floor (fp32 exp2 of log2-scaled arguments is good to ~1e-6 per term; the lse input carries ~5e-6)."""
import numpy as np
import pytest

import oracle
from paper_2609_36301_b200 import binding as mr
from paper_2609_36301_b200 import inputs

from helpers import to_device

pytestmark = pytest.mark.gpu

RTOL, ATOL = 2e-4, 1e-6


def run_psum(case, path):
    import torch
    X, R1, R2 = to_device(case)
    res = mr.route(X, R1, R2, case.k, 1, want_lse=True, path=path)
    psum = torch.full((case.M,), 123.0, dtype=torch.float32, device="cuda")      # must be overwritten
    mr.more_route_psum(X, R1, R2, res.lse, psum, path=path)
    torch.cuda.synchronize()
    assert mr.more_route_status() == 0
    return psum.cpu().numpy().astype(np.float64), res


@pytest.mark.parametrize("T,h,r,M", [(256, 128, 8, 256), (300, 72, 16, 264), (515, 448, 56, 4104), (1000, 256, 32, 2048),
                                      (130, 128, 64, 776), (1, 8, 8, 8)])
def test_psum_tensor_core_path(T, h, r, M):
    case = inputs.gaussian_case(T, h, r, M, min(4, M), 1, seed=61)
    got, _ = run_psum(case, mr.PATH_TCGEN05)
    want, _ = oracle.psum(case.X, case.R1, case.R2)
    np.testing.assert_allclose(got, want, rtol=RTOL, atol=ATOL)
    np.testing.assert_allclose(got.sum(), T, rtol=1e-4)                          # rows of P sum to one


@pytest.mark.parametrize("T,h,r,M", [(33, 40, 8, 130), (300, 100, 12, 1000), (64, 64, 96, 256)])
def test_psum_generic_path(T, h, r, M):
    case = inputs.gaussian_case(T, h, r, M, 2, 1, seed=62)
    got, _ = run_psum(case, mr.PATH_AUTO)
    want, _ = oracle.psum(case.X, case.R1, case.R2)
    np.testing.assert_allclose(got, want, rtol=RTOL, atol=ATOL)


def test_switch_loss_from_counts_and_psum():
    """L_bal = (M/N) f . psum (Eq. app_lbal) from the library's two statistics, mixture inputs (skewed load)."""
    case = inputs.make_config("c3", T=4096)
    got, res = run_psum(case, mr.PATH_AUTO)
    want, _ = oracle.psum(case.X, case.R1, case.R2)
    np.testing.assert_allclose(got, want, rtol=RTOL, atol=ATOL)
    ref = oracle.route(case.X, case.R1, case.R2, case.k, 1)
    f_gpu = res.counts.cpu().numpy() / (case.T * case.k)
    loss_gpu = case.M / case.T * float(f_gpu @ got)
    loss_ref = case.M / case.T * float((ref.counts / (case.T * case.k)) @ want)
    assert abs(loss_gpu - loss_ref) <= 1e-3 * loss_ref
    assert loss_ref > 1.2                                                        # a skewed router is far from balanced


def test_psum_at_the_benchmarked_size():
    """c3 at full size (65536 tokens, 16384 experts: the launch the benchmark's psum line times), every bin against
    the oracle's column sums."""
    case = inputs.make_config("c3")
    got, _ = run_psum(case, mr.PATH_AUTO)
    want, _ = oracle.psum(case.X, case.R1, case.R2)
    np.testing.assert_allclose(got, want, rtol=RTOL, atol=ATOL)
    np.testing.assert_allclose(got.sum(), case.T, rtol=1e-4)
