"""Shared checking code of the GPU parity tests: the acceptance rule, written once.

Acceptance rule (the 1e-3 near-tie exemption and the 2e-3 gate tolerance are the benchmark definition's; the GPU's
logits are good to ~4e-5 because z is carried as a bf16 high part plus a bf16 low part and accumulated in fp32):
  * a token is *exempt* when the oracle's k-th and (k+1)-th logits differ by less than 1e-3;
  * non-exempt tokens: the GPU's set of expert ids equals the oracle's exactly;
  * exempt tokens: ids distinct and in range, every chosen expert's oracle logit >= l_(k) - 1e-3, and every
    expert whose oracle logit exceeds l_(k+1) + 1e-3 is chosen;
  * gates compared position by position in descending order, |diff| <= 2e-3 (and, self-imposed, a relative
    bound, because full-softmax gates are ~1e-3 themselves);
  * counts == bincount(GPU ids) always, and == the oracle's counts when no token's set differs.
"""
from __future__ import annotations

import numpy as np

import oracle
from paper_2609_36301_b200 import inputs

TIE_EPS = 1e-3       # exemption threshold on the oracle's gap l_(k) - l_(k+1)
GATE_ATOL = 2e-3     # absolute gate tolerance of the benchmark definition
GATE_RTOL = 1e-2     # self-imposed relative gate tolerance (on top of a tiny absolute floor)
LSE_ATOL = 1e-3      # self-imposed tolerance on the log-sum-exp
TOPVAL_ATOL = 2e-4   # self-imposed: selected logits vs fp64 (hi+lo bf16 z and fp32 accumulation give ~3e-5)


def to_device(case, device="cuda"):
    import torch
    def dev(a):
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return dev(case.X), dev(case.R1), dev(case.R2)


def check_rows(case, rows, idx, gate, topval=None, lse=None, gate_mode=None, k=None, ref=None):
    """Compare GPU outputs for token ``rows`` (index array into case.X, or None for all) with the oracle.
    Returns a dict of statistics.  ``idx``/``gate``/... are numpy arrays holding just those rows."""
    k = case.k if k is None else k
    gate_mode = case.gate_mode if gate_mode is None else gate_mode
    X = case.X if rows is None else case.X[rows]
    M = case.M
    if ref is None:
        ref = oracle.route(X, case.R1, case.R2, k, gate_mode)
    n = X.shape[0]
    assert idx.shape == (n, k) and gate.shape == (n, k)
    assert idx.min() >= 0 and idx.max() < M, "expert id out of range"
    srt = np.sort(idx, axis=1)
    assert np.all(srt[:, 1:] != srt[:, :-1]), "duplicate expert id within a token"
    exempt = ref.gap < TIE_EPS
    differs = (srt != np.sort(ref.idx, axis=1)).any(axis=1)
    bad = differs & ~exempt
    assert not bad.any(), f"{int(bad.sum())} non-exempt tokens with a wrong expert set (first: {np.flatnonzero(bad)[:5]})"
    # oracle logits of the experts the GPU chose
    chosen = oracle.logits_at(X, case.R1, case.R2, idx)
    kth = ref.topval[:, -1]
    nxt = kth - ref.gap
    if differs.any():
        d = np.flatnonzero(differs)
        assert np.all(chosen[d] >= kth[d, None] - TIE_EPS), "exempt token chose an expert more than 1e-3 below the k-th logit"
        for t in d:
            must = ref.idx[t][ref.topval[t] > nxt[t] + TIE_EPS]
            assert np.isin(must, idx[t]).all(), "exempt token misses an expert clearly above the (k+1)-th logit"
    # listed in descending logit order (allowing swaps of near-equal neighbours)
    assert np.all(np.diff(chosen, axis=1) <= TIE_EPS), "GPU rows are not in descending logit order"
    # gates, position-wise
    gerr = np.abs(gate.astype(np.float64) - ref.gate)
    assert gerr.max() <= GATE_ATOL, f"gate abs error {gerr.max():.3e}"
    rel_ok = gerr <= GATE_RTOL * ref.gate + 1e-7
    assert rel_ok.all(), f"gate relative error too large: {(gerr / ref.gate).max():.3e}"
    stats = dict(tokens=n, exempt=int(exempt.sum()), differs=int(differs.sum()), gate_err=float(gerr.max()))
    if topval is not None:
        terr = np.abs(np.sort(topval.astype(np.float64), axis=1) - np.sort(chosen, axis=1)).max()
        assert terr <= TOPVAL_ATOL, f"selected-logit error {terr:.3e}"
        stats["topval_err"] = float(terr)
    if lse is not None:
        lerr = np.abs(lse.astype(np.float64) - ref.lse).max()
        assert lerr <= LSE_ATOL, f"log-sum-exp error {lerr:.3e}"
        stats["lse_err"] = float(lerr)
    stats["ref"] = ref
    stats["differs_mask"] = differs
    return stats


def check_counts(idx_all, counts, M, ref_counts=None, any_differs=True):
    """counts must be the bincount of the GPU's own ids; and the oracle's when every token's set matched."""
    want = np.bincount(idx_all.ravel().astype(np.int64), minlength=M)
    assert np.array_equal(counts.astype(np.int64), want), "out_counts is not the bincount of out_idx"
    assert counts.sum() == idx_all.size
    if ref_counts is not None and not any_differs:
        assert np.array_equal(counts.astype(np.int64), ref_counts), "out_counts differs from the oracle's"
