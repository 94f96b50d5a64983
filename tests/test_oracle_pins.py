"""Pins of the CPU oracle against things other than itself (no GPU needed).

Each test is chosen so that a plausible mistake in ``oracle/more_oracle.c`` (a dropped term, a wrong sign or
index, a transposed operand, a wrong tie rule, the wrong softmax denominator) fails at least one of them.
"""
import os

import numpy as np
import pytest
from scipy.special import logsumexp, softmax

import oracle
from paper_2609_36301_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------------------------------------
# An independent second implementation: numpy fp64, full T x M matrix, full sort, library softmax.
# --------------------------------------------------------------------------------------------------------
def brute_force(case, k, gate_mode):
    Xd = inputs.bf16_bits_to_f64(case.X)
    R1d = inputs.bf16_bits_to_f64(case.R1)
    R2d = inputs.bf16_bits_to_f64(case.R2)
    L = (Xd @ R1d) @ R2d                                    # Eq. app_logits
    T, M = L.shape
    ids = np.broadcast_to(np.arange(M), (T, M))
    order = np.lexsort((ids, -L), axis=1)[:, :k]            # logit descending, id ascending
    top = np.take_along_axis(L, order, axis=1)
    if gate_mode == 0:
        gate = softmax(top, axis=1)                         # softmax over the k selected (Section 2)
    else:
        gate = np.take_along_axis(softmax(L, axis=1), order, axis=1)   # Eq. app_softmax, selected entries
    counts = np.bincount(order.ravel(), minlength=M)
    return L, order, top, gate, logsumexp(L, axis=1), counts


TINY = [
    # T, h, r, M, k
    (256, 128, 8, 256, 2),     # the tiny benchmark configuration
    (1, 16, 4, 5, 1),          # one token, k = 1, M not a multiple of 8
    (7, 24, 3, 11, 11),        # k == M: every expert selected
    (33, 40, 8, 130, 5),       # ragged everything
    (5, 8, 8, 17, 16),         # k = M - 1
]


@pytest.mark.parametrize("T,h,r,M,k", TINY)
@pytest.mark.parametrize("gate_mode", [0, 1])
def test_matches_numpy_brute_force(T, h, r, M, k, gate_mode):
    case = inputs.gaussian_case(T, h, r, M, k, gate_mode, seed=3)
    res = oracle.route(case.X, case.R1, case.R2, k, gate_mode)
    L, order, top, gate, lse, counts = brute_force(case, k, gate_mode)
    assert np.array_equal(res.idx, order)
    np.testing.assert_allclose(res.topval, top, rtol=0, atol=1e-12)
    np.testing.assert_allclose(res.gate, gate, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(res.lse, lse, rtol=0, atol=1e-12)
    assert np.array_equal(res.counts, counts)
    np.testing.assert_allclose(oracle.logits(case.X, case.R1, case.R2), L, rtol=0, atol=1e-12)
    if k < M:
        srt = -np.sort(-L, axis=1)
        np.testing.assert_allclose(res.gap, srt[:, k - 1] - srt[:, k], rtol=0, atol=1e-12)
    else:
        assert np.all(np.isinf(res.gap))


def test_logits_at_matches_full_matrix():
    case = inputs.gaussian_case(9, 32, 8, 50, 4, 0, seed=5)
    L = oracle.logits(case.X, case.R1, case.R2)
    ids = np.random.default_rng(0).integers(0, 50, size=(9, 6)).astype(np.int32)
    got = oracle.logits_at(case.X, case.R1, case.R2, ids)
    np.testing.assert_allclose(got, np.take_along_axis(L, ids.astype(np.int64), axis=1), rtol=0, atol=1e-13)


# --------------------------------------------------------------------------------------------------------
# Structural invariants and the identity between the two gating modes.
# --------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("shape", [(64, 64, 8, 96, 4), (40, 128, 16, 512, 8)])
def test_invariants_and_mode_identity(shape):
    T, h, r, M, k = shape
    case = inputs.gaussian_case(T, h, r, M, k, 0, seed=11)
    r0 = oracle.route(case.X, case.R1, case.R2, k, 0)
    r1 = oracle.route(case.X, case.R1, case.R2, k, 1)
    assert np.array_equal(r0.idx, r1.idx)
    for res in (r0, r1):
        assert res.idx.min() >= 0 and res.idx.max() < M
        assert all(len(set(row)) == k for row in res.idx.tolist())         # ids distinct
        assert np.all(np.diff(res.topval, axis=1) <= 0)                    # descending logits
        assert np.all(np.diff(res.gate, axis=1) <= 1e-15)                  # hence non-increasing gates
        assert res.counts.sum() == T * k
        assert np.array_equal(res.counts, np.bincount(res.idx.ravel(), minlength=M))
    np.testing.assert_allclose(r0.gate.sum(axis=1), 1.0, atol=1e-12)       # top-k softmax sums to one
    s1 = r1.gate.sum(axis=1)
    assert np.all(s1 > 0) and np.all(s1 <= 1 + 1e-12)                      # a sub-distribution of P
    # P_j / sum_S P = softmax over S;   P_j = exp(l_j - lse)
    np.testing.assert_allclose(r1.gate / s1[:, None], r0.gate, rtol=1e-12)
    np.testing.assert_allclose(r1.gate, np.exp(r1.topval - r1.lse[:, None]), rtol=1e-12)
    # nothing unselected beats something selected
    L = oracle.logits(case.X, case.R1, case.R2)
    mask = np.ones_like(L, dtype=bool)
    np.put_along_axis(mask, r0.idx.astype(np.int64), False, axis=1)
    assert np.all(np.where(mask, L, -np.inf).max(axis=1) <= r0.topval[:, -1])


def test_ties_broken_by_ascending_id():
    # two identical expert columns: the lower id must be listed first, and win the last slot.
    case = inputs.gaussian_case(16, 32, 4, 12, 3, 0, seed=2)
    R2 = case.R2.copy()
    R2[:, 9] = R2[:, 4]
    res = oracle.route(case.X, case.R1, R2, 3, 0)
    for row, vals in zip(res.idx.tolist(), res.topval.tolist()):
        if 4 in row and 9 in row:
            assert row.index(4) + 1 == row.index(9)
        assert not (9 in row and 4 not in row)


# --------------------------------------------------------------------------------------------------------
# Full-rank identity: r = h, R1 = I  ==> the standard router softmax(TopK(R x)) with R = R2^T (Section 2).
# --------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("gate_mode", [0, 1])
def test_full_rank_identity(gate_mode):
    case = inputs.full_rank_case(48, 64, 200, 6, gate_mode, seed=4)
    res = oracle.route(case.X, case.R1, case.R2, 6, gate_mode)
    Rx = inputs.bf16_bits_to_f64(case.X) @ inputs.bf16_bits_to_f64(case.R2)      # R x, no low-rank step at all
    order = np.lexsort((np.broadcast_to(np.arange(200), Rx.shape), -Rx), axis=1)[:, :6]
    assert np.array_equal(res.idx, order)
    top = np.take_along_axis(Rx, order, axis=1)
    want = softmax(top, axis=1) if gate_mode == 0 else np.take_along_axis(softmax(Rx, axis=1), order, axis=1)
    np.testing.assert_allclose(res.gate, want, rtol=1e-12)


# --------------------------------------------------------------------------------------------------------
# Thm. 1 basis construction: the selected set is prescribed; all selected logits tie.
# --------------------------------------------------------------------------------------------------------
def test_thm1_basis_golden():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "thm1_basis_M8_k2.txt")) if not ln.startswith("#")]
    subsets = np.array([[int(a), int(b)] for _, a, b, _, _ in rows])
    for gate_mode, col in ((0, 3), (1, 4)):
        case = inputs.basis_case(subsets, M=8, h=16, gate_mode=gate_mode)
        res = oracle.route(case.X, case.R1, case.R2, 2, gate_mode)
        assert np.array_equal(res.idx, subsets)                          # ties -> ascending id
        np.testing.assert_allclose(res.topval, 1.0, atol=0)
        np.testing.assert_allclose(res.gap, 2.0, atol=0)                 # margin 2 in these units
        want = np.array([[float(rw[col])] * 2 for rw in rows])
        np.testing.assert_allclose(res.gate, want, rtol=1e-14)


def test_thm1_basis_random_subsets():
    rng = np.random.default_rng(7)
    M, h, k, T = 24, 32, 5, 40
    subsets = np.sort(np.array([rng.choice(M, size=k, replace=False) for _ in range(T)]), axis=1)
    case = inputs.basis_case(subsets, M=M, h=h, gate_mode=1)
    res = oracle.route(case.X, case.R1, case.R2, k, 1)
    assert np.array_equal(res.idx, subsets)
    np.testing.assert_allclose(res.gate, np.e / (k * np.e + (M - k) / np.e), rtol=1e-14)
    np.testing.assert_allclose(res.lse, np.log(k * np.e + (M - k) / np.e), rtol=1e-14)


# --------------------------------------------------------------------------------------------------------
# Prop. 1 sign-vector router: closed-form top-2 and uniform k/M marginals.
# --------------------------------------------------------------------------------------------------------
def test_hypercube_closed_form_top2():
    r, T = 8, 256
    case = inputs.hypercube_case(T, 128, r, 2, 0, seed=0)
    res = oracle.route(case.X, case.R1, case.R2, 2, 0)
    x = inputs.bf16_bits_to_f64(case.X)[:, :r]
    a = np.abs(x)
    first = ((x > 0).astype(np.int64) << np.arange(r)).sum(axis=1)       # the sign pattern of z
    weakest = a.argmin(axis=1)
    second = first ^ (1 << weakest)                                      # flip the least-committed coordinate
    assert np.array_equal(res.idx[:, 0], first)
    assert np.array_equal(res.idx[:, 1], second)
    np.testing.assert_allclose(res.topval[:, 0], a.sum(axis=1), rtol=1e-14)
    np.testing.assert_allclose(res.topval[:, 1], a.sum(axis=1) - 2 * a.min(axis=1), rtol=1e-13, atol=1e-14)
    d = 2 * a.min(axis=1)
    np.testing.assert_allclose(res.gate[:, 0], 1 / (1 + np.exp(-d)), rtol=1e-13)
    np.testing.assert_allclose(res.gate[:, 1], 1 / (1 + np.exp(d)), rtol=1e-13)


@pytest.mark.parametrize("k", [1, 3])
def test_hypercube_uniform_marginals_bernstein(k):
    # counts[a] ~ Binomial(T, k/M); Prop. 1's bound at delta = 1e-6.
    r, T = 6, 8192
    M = 1 << r
    case = inputs.hypercube_case(T, 16, r, k, 0, seed=1)
    res = oracle.route(case.X, case.R1, case.R2, k, 0)
    L = np.log(2 * M / 1e-6)
    bound = np.sqrt(2 * T * k * L / M) + 2 * L / 3
    assert np.abs(res.counts - T * k / M).max() <= bound
    assert res.counts.sum() == T * k


# --------------------------------------------------------------------------------------------------------
# Online softmax (Eq. app_online) reproduces the oracle's two-pass (m, Z) for any tiling and tile order.
# --------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("tile", [1, 7, 64, 1000])
def test_online_softmax_recurrence(tile):
    case = inputs.gaussian_case(20, 32, 8, 300, 4, 1, seed=9)
    res = oracle.route(case.X, case.R1, case.R2, 4, 1)
    L = oracle.logits(case.X, case.R1, case.R2)
    starts = list(range(0, 300, tile))
    np.random.default_rng(tile).shuffle(starts)
    m = np.full(20, -np.inf)
    Z = np.zeros(20)
    for s in starts:
        y = L[:, s:s + tile]
        m2 = np.maximum(m, y.max(axis=1))
        Z = Z * np.exp(m - m2) + np.exp(y - m2[:, None]).sum(axis=1)
        m = m2
    np.testing.assert_allclose(m + np.log(Z), res.lse, rtol=0, atol=1e-12)
    np.testing.assert_allclose(np.exp(res.topval - m[:, None]) / Z[:, None], res.gate, rtol=1e-12)


# --------------------------------------------------------------------------------------------------------
# Relabelling experts relabels the selection and changes nothing else (top-k equivariance lemma).
# --------------------------------------------------------------------------------------------------------
def test_expert_permutation_equivariance():
    case = inputs.gaussian_case(32, 48, 8, 77, 5, 1, seed=12)
    perm = np.random.default_rng(1).permutation(77)
    a = oracle.route(case.X, case.R1, case.R2, 5, 1)
    b = oracle.route(case.X, case.R1, case.R2[:, perm], 5, 1)      # new column q holds old expert perm[q]
    assert np.array_equal(perm[b.idx], a.idx)
    np.testing.assert_allclose(b.gate, a.gate, rtol=1e-13)
    np.testing.assert_allclose(b.lse, a.lse, rtol=0, atol=1e-13)
    assert np.array_equal(b.counts, a.counts[perm])


def test_rejects_bad_arguments():
    case = inputs.gaussian_case(4, 8, 2, 6, 2, 0)
    with pytest.raises(ValueError):
        oracle.route(case.X, case.R1, case.R2, 7, 0)      # k > M
    with pytest.raises(ValueError):
        oracle.route(case.X, case.R1, case.R2, 2, 2)      # unknown gate mode


# --------------------------------------------------------------------------------------------------------
# Input recipe: variance matching (sigma_1 sigma_2 = sigma / sqrt r) gives unit-variance logits.
# --------------------------------------------------------------------------------------------------------
def test_generator_gives_unit_variance_logits():
    case = inputs.gaussian_case(64, 512, 16, 2048, 8, 0, seed=0)
    L = oracle.logits(case.X, case.R1, case.R2)
    assert 0.8 < L.var() < 1.25
    # bf16 rounding is round-to-nearest-even and exact on representable values
    f = np.array([1.0, -2.5, 0.0, 1.00390625, 1.01171875], dtype=np.float32)   # last two: ties at bit 16
    back = inputs.bf16_bits_to_f32(inputs.to_bf16_bits(f))
    assert back.tolist() == [1.0, -2.5, 0.0, 1.0, 1.015625]


# --------------------------------------------------------------------------------------------------------
# Dispatch bookkeeping (Sort + Count): a stable counting sort, pinned against numpy's stable argsort.
# --------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("T,k,M", [(1, 1, 1), (7, 3, 5), (64, 4, 1000), (500, 8, 17)])
def test_dispatch_matches_stable_argsort(T, k, M):
    rng = np.random.default_rng(T * 31 + k)
    idx = rng.integers(0, M, size=(T, k)).astype(np.int32)
    offsets, pairs = oracle.dispatch(idx, M)
    flat = idx.ravel()
    assert np.array_equal(pairs, np.argsort(flat, kind="stable"))
    assert np.array_equal(offsets, np.concatenate([[0], np.cumsum(np.bincount(flat, minlength=M))]))
    assert np.all(np.diff(flat[pairs]) >= 0)
    assert offsets[M] == T * k


def test_dispatch_skips_ids_outside_the_expert_range():
    idx = np.array([[0, 9], [2**31 - 1, 1], [1, -3]], dtype=np.int32)
    offsets, pairs = oracle.dispatch(idx, 4)
    assert offsets.tolist() == [0, 1, 3, 3, 3]
    assert pairs.tolist() == [0, 3, 4]


# --------------------------------------------------------------------------------------------------------
# Algorithm 2's statistic psum = column sums of the full softmax (Eq. app_psum) and the Switch loss built on it.
# --------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("T,h,r,M", [(1, 8, 2, 3), (50, 32, 8, 130), (256, 128, 8, 256)])
def test_psum_matches_numpy_softmax_column_sums(T, h, r, M):
    case = inputs.gaussian_case(T, h, r, M, 1, 1, seed=21)
    ps, lse = oracle.psum(case.X, case.R1, case.R2)
    L = (inputs.bf16_bits_to_f64(case.X) @ inputs.bf16_bits_to_f64(case.R1)) @ inputs.bf16_bits_to_f64(case.R2)
    np.testing.assert_allclose(ps, softmax(L, axis=1).sum(axis=0), rtol=1e-12)
    np.testing.assert_allclose(lse, logsumexp(L, axis=1), rtol=0, atol=1e-12)
    np.testing.assert_allclose(ps.sum(), T, rtol=1e-12)                    # every row of P sums to one
    assert np.array_equal(lse, oracle.route(case.X, case.R1, case.R2, 1, 1).lse)   # same row statistics as the router


def test_psum_uniform_router_gives_unit_switch_loss():
    # all-zero expert vectors: P = 1/M everywhere, psum = T/M, and L_bal = (M/N) f . psum = 1 for any dispatch f
    case = inputs.gaussian_case(40, 16, 4, 12, 3, 1, seed=22)
    R2 = np.zeros_like(case.R2)
    ps, _ = oracle.psum(case.X, case.R1, R2)
    np.testing.assert_allclose(ps, 40 / 12, rtol=1e-14)
    res = oracle.route(case.X, case.R1, R2, 3, 1)
    f = res.counts / (40 * 3)
    np.testing.assert_allclose(12 / 40 * (f @ ps), 1.0, rtol=1e-13)
    assert np.array_equal(res.idx, np.broadcast_to(np.arange(3), (40, 3)))  # exact ties everywhere: lowest ids


def test_psum_is_equivariant_under_expert_relabelling():
    case = inputs.gaussian_case(30, 24, 6, 41, 2, 1, seed=23)
    perm = np.random.default_rng(3).permutation(41)
    a, _ = oracle.psum(case.X, case.R1, case.R2)
    b, _ = oracle.psum(case.X, case.R1, case.R2[:, perm])
    np.testing.assert_allclose(b, a[perm], rtol=1e-13)


# ------------------------------------------------------------------------------------------- shard merge
def _shard_partials(case, bounds, k):
    """Oracle routes of the expert ranges [bounds[s], bounds[s+1]) with ids made global; k_s = min(k, shard size)."""
    S = len(bounds) - 1
    T = case.X.shape[0]
    idx = np.full((S, T, k), -1, dtype=np.int32)
    val = np.full((S, T, k), -np.inf)
    lse = np.zeros((S, T))
    for s in range(S):
        lo, hi = bounds[s], bounds[s + 1]
        ks = min(k, hi - lo)
        ref = oracle.route(case.X, case.R1, np.ascontiguousarray(case.R2[:, lo:hi]), ks, 1)
        idx[s, :, :ks] = ref.idx + lo
        val[s, :, :ks] = ref.topval
        lse[s] = ref.lse
    return idx, val, lse


@pytest.mark.parametrize("gate_mode", [0, 1])
@pytest.mark.parametrize("bounds", [(0, 96), (0, 48, 96), (0, 8, 40, 41, 96), (0, 3, 96)])
def test_merge_of_expert_shards_equals_the_unsharded_route(bounds, gate_mode):
    """A global top-k member is a top-k member of its own shard, and the shards' (m, Z) pairs combine like tiles in
    Eq. app_online: merging the per-shard routes must reproduce the route over all experts (plain definition)."""
    k = 6
    case = inputs.gaussian_case(64, 32, 8, 96, k, gate_mode, seed=11)
    full = oracle.route(case.X, case.R1, case.R2, k, gate_mode)
    idx, val, lse = _shard_partials(case, bounds, k)
    m_idx, m_gate, m_val, m_lse, m_counts = oracle.merge(idx, val, lse, 96, gate_mode)
    assert np.array_equal(m_idx, full.idx)
    np.testing.assert_allclose(m_val, full.topval, rtol=0, atol=0)          # the same fp64 numbers, only re-ordered
    np.testing.assert_allclose(m_gate, full.gate, rtol=1e-12, atol=0)
    np.testing.assert_allclose(m_lse, full.lse, rtol=1e-13, atol=1e-13)
    assert np.array_equal(m_counts, full.counts)


def test_merge_breaks_ties_by_ascending_id_and_ignores_unused_slots():
    # two shards, one token, k = 3; equal logits 2.0 at ids 7 (shard 1) and 4 (shard 0): 4 goes first
    idx = np.array([[[4, 1, -1]], [[7, 9, 8]]], dtype=np.int32)
    val = np.array([[[2.0, 0.5, 123.0]], [[2.0, 3.0, -1.0]]])
    m_idx, m_gate, m_val, m_lse, counts = oracle.merge(idx, val, None, 10, 0)
    assert m_idx.tolist() == [[9, 4, 7]]
    e = np.exp(np.array([3.0, 2.0, 2.0]) - 3.0)
    np.testing.assert_allclose(m_gate[0], e / e.sum(), rtol=1e-15)
    assert m_lse is None and counts.tolist() == [0, 0, 0, 0, 1, 0, 0, 1, 0, 1]
    # fewer valid pairs than k: the tail is (-1, gate 0)
    idx2 = np.array([[[5, -1, -1]]], dtype=np.int32)
    val2 = np.array([[[1.0, 0.0, 0.0]]])
    m_idx2, m_gate2, _, _, counts2 = oracle.merge(idx2, val2, None, 6, 0)
    assert m_idx2.tolist() == [[5, -1, -1]] and m_gate2.tolist() == [[1.0, 0.0, 0.0]] and counts2.sum() == 1
    with pytest.raises(ValueError):
        oracle.merge(idx, val, None, 10, 1)                                  # full-softmax gates need the lse
