"""Seeded synthetic inputs for the low-rank router, shared by the CUDA path's tests/bench and the CPU oracle's tests.

This module only *draws numbers and lays them out*; it contains none of the router's arithmetic
(no projection, no logits, no top-k, no softmax).  Everything is generated in fp32 on the host from a
counter-based generator (numpy Philox keyed by ``(seed, stream)``), rounded to bfloat16 once
(round-to-nearest-even) and returned as ``uint16`` bit patterns, so the GPU library and the oracle read
byte-identical operands.

Operand naming follows the library's C interface: ``X [T][h]``, ``R1 [h][r]`` (down-projection, the paper's
R_2 transposed), ``R2 [r][M]`` (expert vectors as columns, the paper's R_1 transposed); all row-major.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

# Sub-stream ids of the generator (one independent Philox stream per tensor).
STREAM_X, STREAM_R1, STREAM_R2, STREAM_MEANS, STREAM_ASSIGN, STREAM_MISC = 1, 2, 3, 4, 5, 6


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=np.array([seed, stream], dtype=np.uint64)))


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """fp32 -> bfloat16 bit pattern (uint16), round-to-nearest-even; finite inputs only."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bfloat16 bit pattern (uint16) -> the fp32 value it denotes (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


@dataclass
class RouterCase:
    """One router problem: bf16 operands as uint16 bit patterns plus its shape."""
    name: str
    X: np.ndarray   # [T][h] uint16
    R1: np.ndarray  # [h][r] uint16
    R2: np.ndarray  # [r][M] uint16
    k: int
    gate_mode: int
    meta: dict = field(default_factory=dict)

    @property
    def T(self) -> int:
        return self.X.shape[0]

    @property
    def h(self) -> int:
        return self.X.shape[1]

    @property
    def r(self) -> int:
        return self.R1.shape[1]

    @property
    def M(self) -> int:
        return self.R2.shape[1]


def _normal_bf16(rng: np.random.Generator, shape, scale: float, chunk_rows: int = 8192) -> np.ndarray:
    """N(0, scale^2) samples of ``shape`` as bf16 bits, drawn row-chunk by row-chunk (same stream order)."""
    rows = shape[0]
    out = np.empty(shape, dtype=np.uint16)
    for lo in range(0, rows, chunk_rows):
        hi = min(rows, lo + chunk_rows)
        blk = rng.standard_normal((hi - lo,) + tuple(shape[1:]), dtype=np.float32)
        if scale != 1.0:
            blk *= np.float32(scale)
        out[lo:hi] = to_bf16_bits(blk)
    return out


def router_weights(h: int, r: int, M: int, seed: int = 0):
    """R1 ~ N(0, 1/h), R2 ~ N(0, 1/r) i.i.d., so that logits of a unit-variance token have variance ~1."""
    R1 = _normal_bf16(_rng(seed, STREAM_R1), (h, r), 1.0 / np.sqrt(h))
    R2 = _normal_bf16(_rng(seed, STREAM_R2), (r, M), 1.0 / np.sqrt(r))
    return R1, R2


def gaussian_case(T: int, h: int, r: int, M: int, k: int, gate_mode: int, seed: int = 0,
                  name: str = "gaussian") -> RouterCase:
    """X ~ N(0,1) i.i.d.; weights from :func:`router_weights`."""
    X = _normal_bf16(_rng(seed, STREAM_X), (T, h), 1.0)
    R1, R2 = router_weights(h, r, M, seed)
    return RouterCase(name, X, R1, R2, k, gate_mode, {"seed": seed, "dist": "gaussian"})


def mixture_case(T: int, h: int, r: int, M: int, k: int, gate_mode: int, seed: int = 0,
                 components: int = 64, within_sd: float = 0.5, name: str = "mixture") -> RouterCase:
    """X rows from a ``components``-component Gaussian mixture (means ~ N(0,I), sd ``within_sd``, uniform
    component weights): tokens of one component share favourite experts, which skews the expert load."""
    means = _rng(seed, STREAM_MEANS).standard_normal((components, h), dtype=np.float32)
    assign = _rng(seed, STREAM_ASSIGN).integers(0, components, size=T, dtype=np.int64)
    rng = _rng(seed, STREAM_X)
    X = np.empty((T, h), dtype=np.uint16)
    chunk = 8192
    for lo in range(0, T, chunk):
        hi = min(T, lo + chunk)
        blk = rng.standard_normal((hi - lo, h), dtype=np.float32)
        blk *= np.float32(within_sd)
        blk += means[assign[lo:hi]]
        X[lo:hi] = to_bf16_bits(blk)
    R1, R2 = router_weights(h, r, M, seed)
    return RouterCase(name, X, R1, R2, k, gate_mode,
                      {"seed": seed, "dist": "mixture", "components": components, "assign": assign})


def hypercube_case(T: int, h: int, r: int, k: int, gate_mode: int, seed: int = 0) -> RouterCase:
    """Sign-vector router on M = 2^r experts: R1 = [I_r; 0] selects the first r coordinates and column ``a``
    of R2 is the +-1 pattern whose bit l (LSB first) is set iff coordinate l is +1.  All entries are
    exactly representable in bf16."""
    assert h >= r and r <= 16
    M = 1 << r
    X = _normal_bf16(_rng(seed, STREAM_X), (T, h), 1.0)
    R1f = np.zeros((h, r), dtype=np.float32)
    R1f[np.arange(r), np.arange(r)] = 1.0
    a = np.arange(M, dtype=np.int64)
    bits = (a[None, :] >> np.arange(r, dtype=np.int64)[:, None]) & 1      # [r][M]
    R2f = (2.0 * bits - 1.0).astype(np.float32)
    return RouterCase("hypercube", X, to_bf16_bits(R1f), to_bf16_bits(R2f), k, gate_mode,
                      {"seed": seed, "dist": "hypercube"})


def basis_case(subsets: np.ndarray, M: int, h: int, gate_mode: int) -> RouterCase:
    """Uncompressed basis router: r = M <= h, R1 = [I_M; 0], R2 = I_M; token n is +1 on ``subsets[n]`` and -1
    on the other experts' coordinates (0 beyond M), so its k selected experts are prescribed."""
    subsets = np.asarray(subsets, dtype=np.int64)
    T, k = subsets.shape
    assert M <= h
    Xf = np.zeros((T, h), dtype=np.float32)
    Xf[:, :M] = -1.0
    Xf[np.arange(T)[:, None], subsets] = 1.0
    R1f = np.zeros((h, M), dtype=np.float32)
    R1f[np.arange(M), np.arange(M)] = 1.0
    R2f = np.eye(M, dtype=np.float32)
    return RouterCase("basis", to_bf16_bits(Xf), to_bf16_bits(R1f), to_bf16_bits(R2f), k, gate_mode,
                      {"dist": "basis"})


def full_rank_case(T: int, h: int, M: int, k: int, gate_mode: int, seed: int = 0) -> RouterCase:
    """r = h with R1 = I_h: the low-rank router degenerates to the standard router with R = R2^T."""
    X = _normal_bf16(_rng(seed, STREAM_X), (T, h), 1.0)
    R1f = np.eye(h, dtype=np.float32)
    R2 = _normal_bf16(_rng(seed, STREAM_R2), (h, M), 1.0 / np.sqrt(h))
    return RouterCase("full_rank", X, to_bf16_bits(R1f), R2, k, gate_mode, {"seed": seed, "dist": "full_rank"})


GATE_TOPK_SOFTMAX = 0
GATE_FULL_SOFTMAX = 1

# The benchmark configurations (shape, k, default gate mode, input recipe).
CONFIGS = {
    "c0":        dict(T=256,   h=128,  r=8,  M=256,    k=2,  gate_mode=0, dist="gaussian"),
    "c1":        dict(T=16384, h=512,  r=16, M=4096,   k=8,  gate_mode=1, dist="gaussian"),
    "c2_M1024":  dict(T=32768, h=512,  r=32, M=1024,   k=8,  gate_mode=0, dist="gaussian"),
    "c2_M4096":  dict(T=32768, h=512,  r=32, M=4096,   k=8,  gate_mode=0, dist="gaussian"),
    "c2_M16384": dict(T=32768, h=512,  r=32, M=16384,  k=8,  gate_mode=0, dist="gaussian"),
    "c2_M65536": dict(T=32768, h=512,  r=32, M=65536,  k=8,  gate_mode=0, dist="gaussian"),
    "c3":        dict(T=65536, h=2048, r=64, M=16384,  k=8,  gate_mode=0, dist="mixture"),
    "c4":        dict(T=8192,  h=4096, r=64, M=131072, k=16, gate_mode=1, dist="gaussian"),
}


def make_config(name: str, seed: int = 0, gate_mode: int | None = None, T: int | None = None) -> RouterCase:
    """Build one of :data:`CONFIGS`; ``T`` may be lowered to get a shorter prefix-shaped sample of the same recipe."""
    c = dict(CONFIGS[name])
    dist = c.pop("dist")
    if gate_mode is not None:
        c["gate_mode"] = gate_mode
    if T is not None:
        c["T"] = T
    if dist == "mixture":
        return mixture_case(seed=seed, name=name, **c)
    return gaussian_case(seed=seed, name=name, **c)
