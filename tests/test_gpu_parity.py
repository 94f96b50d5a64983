"""Parity of the CUDA router (through the C interface) with the CPU oracle, element by element, on a B200."""
import numpy as np
import pytest

import oracle
from paper_2609_36301_b200 import binding as mr
from paper_2609_36301_b200 import inputs

from helpers import check_counts, check_rows, to_device

pytestmark = pytest.mark.gpu


def run_gpu(case, k=None, gate_mode=None, path=mr.PATH_AUTO, msplit=0):
    import torch
    k = case.k if k is None else k
    gate_mode = case.gate_mode if gate_mode is None else gate_mode
    X, R1, R2 = to_device(case)
    res = mr.route(X, R1, R2, k, gate_mode, want_topval=True, want_lse=True, path=path, msplit=msplit)
    torch.cuda.synchronize()
    assert mr.more_route_status() == 0
    return (res.idx.cpu().numpy(), res.gate.cpu().numpy(), res.counts.cpu().numpy(), res.topval.cpu().numpy(),
            res.lse.cpu().numpy())


def full_check(case, path=mr.PATH_AUTO, msplit=0, k=None, gate_mode=None):
    idx, gate, counts, topval, lse = run_gpu(case, k, gate_mode, path, msplit)
    st = check_rows(case, None, idx, gate, topval, lse, gate_mode=gate_mode, k=k)
    check_counts(idx, counts, case.M, st["ref"].counts, any_differs=bool(st["differs_mask"].any()))
    return st


# ------------------------------------------------------------------------------------------------------------
# tiny configuration, both gating modes, both paths, with and without an expert split
# ------------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("gate_mode", [0, 1])
@pytest.mark.parametrize("path,msplit", [(mr.PATH_GENERIC, 0), (mr.PATH_TCGEN05, 1), (mr.PATH_TCGEN05, 2)])
def test_c0_tiny(gate_mode, path, msplit):
    case = inputs.make_config("c0", gate_mode=gate_mode)
    full_check(case, path, msplit)


# shapes the tensor-core path cannot take (odd h / r / M): generic kernels
@pytest.mark.parametrize("T,h,r,M,k", [(1, 16, 4, 5, 1), (7, 24, 3, 11, 11), (33, 40, 8, 130, 5), (5, 8, 8, 17, 16),
                                        (300, 100, 12, 1000, 32), (64, 64, 96, 256, 4)])
@pytest.mark.parametrize("gate_mode", [0, 1])
def test_generic_path_odd_shapes(T, h, r, M, k, gate_mode):
    case = inputs.gaussian_case(T, h, r, M, k, gate_mode, seed=21)
    assert mr.more_route_plan(T, h, r, M, k).path == mr.PATH_GENERIC
    full_check(case)


# ragged tokens / experts / ranks on the tensor-core path: several tiles plus a tail in every dimension
TC_SHAPES = [
    # T,   h,   r,  M,    k
    (1,    8,   8,  8,    1),
    (129,  64,  8,  136,  2),
    (200,  72,  16, 264,  8),
    (384,  520, 24, 1000, 8),
    (257,  256, 32, 2048, 16),
    (130,  128, 40, 776,  32),
    (256,  192, 64, 1544, 8),
    (515,  448, 56, 4104, 5),
]


@pytest.mark.parametrize("T,h,r,M,k", TC_SHAPES)
@pytest.mark.parametrize("gate_mode", [0, 1])
def test_tcgen05_ragged_shapes(T, h, r, M, k, gate_mode):
    case = inputs.gaussian_case(T, h, r, M, k, gate_mode, seed=31)
    assert mr.more_route_plan(T, h, r, M, k).path == mr.PATH_TCGEN05
    full_check(case, mr.PATH_TCGEN05, 1)


@pytest.mark.parametrize("msplit", [2, 3, 5])
def test_expert_split_gives_identical_results(msplit):
    """Results must not depend on how the expert range is cut across CTAs (block sizes are free parameters of
    Algorithm 1)."""
    case = inputs.gaussian_case(300, 256, 32, 4096, 8, 1, seed=5)
    base = run_gpu(case, path=mr.PATH_TCGEN05, msplit=1)
    other = run_gpu(case, path=mr.PATH_TCGEN05, msplit=msplit)
    assert np.array_equal(base[0], other[0])
    assert np.array_equal(base[2], other[2])
    assert np.array_equal(base[3], other[3])                      # selected logits: same arithmetic, bit-exact
    np.testing.assert_allclose(base[1], other[1], rtol=1e-5, atol=1e-7)
    np.testing.assert_allclose(base[4], other[4], rtol=0, atol=1e-5)
    full_check(case, mr.PATH_TCGEN05, msplit)


def test_paths_agree_on_device():
    case = inputs.gaussian_case(1024, 512, 32, 8192, 8, 1, seed=9)
    a = run_gpu(case, path=mr.PATH_GENERIC)
    b = run_gpu(case, path=mr.PATH_TCGEN05)
    differ = (np.sort(a[0], 1) != np.sort(b[0], 1)).any(axis=1)
    assert differ.mean() < 2e-3
    np.testing.assert_allclose(a[3][~differ], b[3][~differ], rtol=0, atol=2e-4)
    np.testing.assert_allclose(a[4], b[4], rtol=0, atol=1e-4)


# ------------------------------------------------------------------------------------------------------------
# closed-form fixtures
# ------------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("path", [mr.PATH_GENERIC, mr.PATH_TCGEN05])
def test_hypercube_router_closed_form(path):
    """Prop. 1 sign-vector router: top-1 is the sign pattern of the first r coordinates, the runner-up flips the
    least-committed coordinate; gates are sigmoid(+-2 min|x|)."""
    r = 8
    case = inputs.hypercube_case(256, 128, r, 2, 0, seed=0)
    idx, gate, counts, topval, lse = run_gpu(case, path=path)
    x = inputs.bf16_bits_to_f64(case.X)[:, :r]
    a = np.abs(x)
    first = ((x > 0).astype(np.int64) << np.arange(r)).sum(axis=1)
    second = first ^ (1 << a.argmin(axis=1))
    assert np.array_equal(idx[:, 0], first)
    clear = 2 * a.min(axis=1) > 1e-3                  # the runner-up is unique when the smallest |x| is not tiny ...
    srt = np.sort(a, axis=1)
    clear &= (srt[:, 1] - srt[:, 0]) * 2 > 1e-3       # ... and the third-best is clearly behind
    assert np.array_equal(idx[clear, 1], second[clear])
    np.testing.assert_allclose(topval[:, 0], a.sum(axis=1), rtol=0, atol=1e-4)
    np.testing.assert_allclose(gate[:, 0], 1 / (1 + np.exp(-2 * a.min(axis=1))), rtol=0, atol=1e-4)
    full_check(case, path)


@pytest.mark.parametrize("gate_mode", [0, 1])
def test_basis_router_prescribed_sets(gate_mode):
    """Thm. 1 construction in the uncompressed regime: the selected set is prescribed and all selected logits tie."""
    rng = np.random.default_rng(3)
    M, h, k, T = 64, 64, 6, 200
    subsets = np.sort(np.array([rng.choice(M, size=k, replace=False) for _ in range(T)]), axis=1)
    case = inputs.basis_case(subsets, M=M, h=h, gate_mode=gate_mode)
    idx, gate, counts, topval, lse = run_gpu(case, path=mr.PATH_TCGEN05)
    assert np.array_equal(idx, subsets)                       # exact ties: ascending id
    assert np.all(topval == 1.0)
    want = 1.0 / k if gate_mode == 0 else np.e / (k * np.e + (M - k) / np.e)
    np.testing.assert_allclose(gate, want, rtol=1e-5)
    assert np.array_equal(counts, np.bincount(subsets.ravel(), minlength=M))


@pytest.mark.parametrize("gate_mode", [0, 1])
def test_full_rank_identity(gate_mode):
    """r = h, R1 = I: the low-rank router must reproduce the standard router softmax(TopK(R x))."""
    case = inputs.full_rank_case(300, 64, 1024, 8, gate_mode, seed=4)
    full_check(case, mr.PATH_TCGEN05, 1)


def test_duplicate_expert_columns_tie_break():
    case = inputs.gaussian_case(256, 64, 16, 256, 4, 0, seed=2)
    case.R2[:, 200] = case.R2[:, 17]
    case.R2[:, 130] = case.R2[:, 17]
    for path in (mr.PATH_GENERIC, mr.PATH_TCGEN05):
        idx, *_ = run_gpu(case, path=path)
        ref = oracle.route(case.X, case.R1, case.R2, 4, 0)
        assert np.array_equal(np.sort(idx, 1)[ref.gap >= 1e-3], np.sort(ref.idx, 1)[ref.gap >= 1e-3])
        for row in idx.tolist():
            got = [e for e in row if e in (17, 130, 200)]
            assert got == sorted(got) and got == [17, 130, 200][:len(got)]   # lower ids first, and chosen first


# ------------------------------------------------------------------------------------------------------------
# API behaviour on the device
# ------------------------------------------------------------------------------------------------------------
def test_zero_tokens_and_counts_overwritten():
    import torch
    case = inputs.gaussian_case(8, 64, 16, 256, 2, 0)
    X, R1, R2 = to_device(case)
    counts = torch.full((256,), 77, dtype=torch.int32, device="cuda")
    idx = torch.empty((0, 2), dtype=torch.int32, device="cuda")
    gate = torch.empty((0, 2), dtype=torch.float32, device="cuda")
    mr.more_route(X[:0], R1, R2, 2, 0, idx, gate, counts)
    torch.cuda.synchronize()
    assert int(counts.abs().sum()) == 0
    counts.fill_(5)
    idx = torch.empty((8, 2), dtype=torch.int32, device="cuda")
    gate = torch.empty((8, 2), dtype=torch.float32, device="cuda")
    mr.more_route(X, R1, R2, 2, 0, idx, gate, counts)
    torch.cuda.synchronize()
    assert int(counts.sum()) == 16


def test_host_entry_point_matches_device_entry_point():
    import torch
    case = inputs.gaussian_case(500, 128, 16, 1024, 4, 1, seed=8)
    dev = run_gpu(case)
    idx = np.empty((500, 4), dtype=np.int32)
    gate = np.empty((500, 4), dtype=np.float32)
    counts = np.empty((1024,), dtype=np.int32)
    mr.more_route_host(case.X, case.R1, case.R2, 4, 1, idx, gate, counts)
    assert np.array_equal(idx, dev[0]) and np.array_equal(counts, dev[2])
    assert np.array_equal(gate, dev[1])
    # pinned torch tensors work as well
    Xp = torch.from_numpy(case.X.view(np.int16)).pin_memory()
    idx_p = torch.empty((500, 4), dtype=torch.int32).pin_memory()
    gate_p = torch.empty((500, 4), dtype=torch.float32).pin_memory()
    counts_p = torch.empty((1024,), dtype=torch.int32).pin_memory()
    mr.more_route_host(Xp, case.R1, case.R2, 4, 1, idx_p, gate_p, counts_p)
    assert np.array_equal(idx_p.numpy(), dev[0])


def test_non_default_stream_and_repeat_calls():
    import torch
    case = inputs.gaussian_case(1000, 256, 32, 2048, 8, 0, seed=6)
    X, R1, R2 = to_device(case)
    s = torch.cuda.Stream()
    outs = []
    with torch.cuda.stream(s):
        for _ in range(3):
            outs.append(mr.route(X, R1, R2, 8, 0, stream=s))
    s.synchronize()
    for o in outs[1:]:
        assert torch.equal(o.idx, outs[0].idx) and torch.equal(o.counts, outs[0].counts)
        assert torch.equal(o.gate, outs[0].gate)
    assert mr.more_route_status(s) == 0
    assert mr.launches() > 0


def test_k_equals_m_on_tensor_core_path():
    """Every expert selected (k == M): the list is the whole sorted row."""
    case = inputs.gaussian_case(200, 64, 16, 16, 16, 1, seed=12)
    assert mr.more_route_plan(200, 64, 16, 16, 16).path == mr.PATH_TCGEN05
    idx, gate, counts, topval, lse = run_gpu(case, path=mr.PATH_TCGEN05)
    assert np.array_equal(np.sort(idx, axis=1), np.broadcast_to(np.arange(16), (200, 16)))
    assert np.all(counts == 200)
    np.testing.assert_allclose(gate.sum(axis=1), 1.0, atol=1e-5)       # P over all experts sums to one
    full_check(case, mr.PATH_TCGEN05, 1)


def test_sorted_ascending_logits_worst_case_for_the_running_threshold():
    """Experts ordered so that every token's logits increase with the expert id: every new column beats the running
    threshold, the worst case for the candidate buffers (they overflow constantly)."""
    case = inputs.gaussian_case(256, 64, 8, 1024, 8, 0, seed=13)
    # make all logits of a token increase with the expert id: z has one positive component, R2 is a ramp
    R1f = np.zeros((64, 8), dtype=np.float32); R1f[0, 0] = 1.0
    Xf = inputs.bf16_bits_to_f32(case.X); Xf[:, 0] = np.abs(Xf[:, 0]) + 0.5
    R2f = np.zeros((8, 1024), dtype=np.float32); R2f[0] = np.arange(1024, dtype=np.float32) / 128.0
    case.X, case.R1, case.R2 = inputs.to_bf16_bits(Xf), inputs.to_bf16_bits(R1f), inputs.to_bf16_bits(R2f)
    for path in (mr.PATH_TCGEN05, mr.PATH_GENERIC):
        idx, *_ = run_gpu(case, path=path)
        ref = oracle.route(case.X, case.R1, case.R2, 8, 0)
        assert np.array_equal(idx, ref.idx)            # bf16 ramp has exact ties: ids ascending within ties


def test_non_finite_inputs_terminate_and_leave_other_tokens_alone():
    import torch
    case = inputs.gaussian_case(300, 64, 16, 512, 4, 1, seed=14)
    Xf = inputs.bf16_bits_to_f32(case.X)
    Xf[7, :] = np.nan
    Xf[130, 3] = np.inf
    bad = inputs.to_bf16_bits(np.nan_to_num(Xf, nan=0.0, posinf=0.0))
    bad[7, :] = 0x7FC0            # bf16 quiet NaN
    bad[130, 3] = 0x7F80          # +inf
    clean = inputs.to_bf16_bits(np.nan_to_num(Xf, nan=0.0, posinf=0.0))
    for path in (mr.PATH_TCGEN05, mr.PATH_GENERIC):
        case.X = bad
        got = run_gpu(case, path=path)                       # must return; status checked inside run_gpu
        case.X = clean
        want = run_gpu(case, path=path)
        keep = np.ones(300, dtype=bool); keep[[7, 130]] = False
        assert np.array_equal(got[0][keep], want[0][keep])   # rows without bad values are unaffected
        assert got[2].sum() <= 300 * 4 and got[2].min() >= 0
