"""Thin ctypes binding of ``libmore_route.so``: argument marshalling only.

Every step of the router runs in the library's CUDA kernels; torch is used for device memory and streams.
There is no CPU fallback: if the shared library is missing the import of a routing call raises.
The C interface and its semantics are documented in ``include/more_route.h``.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

from . import build as _build

GATE_TOPK_SOFTMAX = 0
GATE_FULL_SOFTMAX = 1
PATH_AUTO, PATH_GENERIC, PATH_TCGEN05 = 0, 1, 2
K_MAX = 32

_lib = None


class MoreRouteError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what} failed: {code} ({strerror(code)})")
        self.code = code


def lib() -> ctypes.CDLL:
    """Load (once) the in-tree shared library; raises if it has not been built.  ``MORE_ROUTE_LIB`` names another
    build of the same sources to load instead (the diagnostic builds of ``build.py``)."""
    global _lib
    if _lib is None:
        path = os.environ.get("MORE_ROUTE_LIB") or _build.LIB_PATH
        if not os.path.exists(path):
            raise FileNotFoundError(
                f"{path} is missing: build it with `python -m paper_2609_36301_b200.build` "
                "(there is no fallback implementation)")
        L = ctypes.CDLL(path)
        vp, i32 = ctypes.c_void_p, ctypes.c_int
        L.more_route.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp]
        L.more_route.restype = i32
        L.more_route_ex.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, i32, i32, vp]
        L.more_route_ex.restype = i32
        L.more_route_host.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp]
        L.more_route_host.restype = i32
        L.more_route_psum.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp, vp, i32, vp]
        L.more_route_psum.restype = i32
        L.more_dispatch.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp]
        L.more_dispatch.restype = i32
        L.more_route_full.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, i32, vp]
        L.more_route_full.restype = i32
        L.more_merge_shards.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp]
        L.more_merge_shards.restype = i32
        L.more_route_noalloc.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp]
        L.more_route_noalloc.restype = i32
        L.more_route_noalloc_capacity.argtypes = []
        L.more_route_noalloc_capacity.restype = ctypes.c_longlong
        ip = ctypes.POINTER(ctypes.c_int)
        L.more_route_plan.argtypes = [i32, i32, i32, i32, i32, i32, i32, i32, ip, ip, ip]
        L.more_route_plan.restype = i32
        L.more_route_plan_ex.argtypes = [i32, i32, i32, i32, i32, i32, i32, i32, i32, ip]
        L.more_route_plan_ex.restype = i32
        L.more_route_status.argtypes = [vp]
        L.more_route_status.restype = i32
        L.more_route_launches.argtypes = []
        L.more_route_launches.restype = ctypes.c_longlong
        # diagnostics (csrc/more_debug.h; not part of the public interface)
        L.more_debug_expire_wait.argtypes = [ctypes.c_longlong, vp]
        L.more_debug_expire_wait.restype = i32
        L.more_debug_scratch_guard.argtypes = [vp]
        L.more_debug_scratch_guard.restype = i32
        L.more_strerror.argtypes = [i32]
        L.more_strerror.restype = ctypes.c_char_p
        L.more_version.argtypes = []
        L.more_version.restype = i32
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().more_strerror(code).decode()


def version() -> int:
    return lib().more_version()


def launches() -> int:
    return int(lib().more_route_launches())


@dataclass
class RoutePlan:
    path: int
    msplit: int
    ctas: int
    block_tokens: int = 0
    token_groups: int = 1
    expert_ranges: int = 1
    filter: bool = False
    paired: bool = False


def more_route_plan(T, h, r, M, k, gate_mode=0, path=PATH_AUTO, msplit=0) -> RoutePlan:
    a, b, c = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    rc = lib().more_route_plan(T, h, r, M, k, gate_mode, path, msplit, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c))
    if rc != 0:
        raise MoreRouteError(rc, "more_route_plan")
    return RoutePlan(a.value, b.value, c.value)


def more_route_plan_ex(T, h, r, M, k, gate_mode=0, want_lse=False, path=PATH_AUTO, msplit=0) -> RoutePlan:
    o = (ctypes.c_int * 8)()
    rc = lib().more_route_plan_ex(T, h, r, M, k, gate_mode, int(want_lse), path, msplit, o)
    if rc != 0:
        raise MoreRouteError(rc, "more_route_plan_ex")
    return RoutePlan(o[0], o[1], o[2], o[3], o[4], o[5], bool(o[6]), bool(o[7]))


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def more_route(X, R1, R2, k, gate_mode, out_idx, out_gate, out_counts, stream=None):
    """``more_route`` of the C interface on torch CUDA tensors (bf16 ``X [T,h]``, ``R1 [h,r]``, ``R2 [r,M]``; int32
    ``out_idx [T,k]``, fp32 ``out_gate [T,k]``, int32 ``out_counts [M]``).  Asynchronous on ``stream``."""
    T, h = X.shape
    r, M = R2.shape
    rc = lib().more_route(_ptr(X), _ptr(R1), _ptr(R2), T, h, r, M, k, gate_mode,
                          _ptr(out_idx), _ptr(out_gate), _ptr(out_counts), _stream(stream))
    if rc != 0:
        raise MoreRouteError(rc, "more_route")


def more_route_ex(X, R1, R2, k, gate_mode, out_idx, out_gate, out_counts, out_topval=None, out_lse=None,
                  path=PATH_AUTO, msplit=0, stream=None):
    """``more_route_ex`` of the C interface (optional selected logits / log-sum-exp outputs, forced path and split)."""
    T, h = X.shape
    r, M = R2.shape
    rc = lib().more_route_ex(_ptr(X), _ptr(R1), _ptr(R2), T, h, r, M, k, gate_mode,
                             _ptr(out_idx), _ptr(out_gate), _ptr(out_counts), _ptr(out_topval), _ptr(out_lse),
                             path, msplit, _stream(stream))
    if rc != 0:
        raise MoreRouteError(rc, "more_route_ex")


def more_route_host(X, R1, R2, k, gate_mode, out_idx, out_gate, out_counts, stream=None):
    """``more_route_host`` on HOST tensors or numpy arrays (``X``/``R1``/``R2`` as bf16 tensors or uint16 arrays);
    copies in, routes, copies out and synchronises before returning."""
    def hp(a):
        return ctypes.c_void_p(a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data)
    T, h = X.shape
    r, M = R2.shape
    rc = lib().more_route_host(hp(X), hp(R1), hp(R2), T, h, r, M, k, gate_mode, hp(out_idx), hp(out_gate),
                               hp(out_counts), _stream(stream))
    if rc != 0:
        raise MoreRouteError(rc, "more_route_host")


def more_route_noalloc(X, R1, R2, k, gate_mode, out_idx, out_gate, out_counts, stream=None):
    """``more_route_noalloc`` of the C interface: same arguments as :func:`more_route`; the library allocates nothing
    (its scratch is a fixed array inside the library image) and rejects ``T * r`` beyond
    :func:`more_route_noalloc_capacity` with ``MORE_ERR_TOO_LARGE``.  For callers that may not use the CUDA allocator."""
    T, h = X.shape
    r, M = R2.shape
    rc = lib().more_route_noalloc(_ptr(X), _ptr(R1), _ptr(R2), T, h, r, M, k, gate_mode,
                                  _ptr(out_idx), _ptr(out_gate), _ptr(out_counts), _stream(stream))
    if rc != 0:
        raise MoreRouteError(rc, "more_route_noalloc")


def more_route_noalloc_capacity() -> int:
    return int(lib().more_route_noalloc_capacity())


def more_route_psum(X, R1, R2, lse, out_psum, path=PATH_AUTO, stream=None):
    """``more_route_psum`` of the C interface: ``out_psum [M]`` (fp32, overwritten) = column sums of the softmax over
    all experts, given every token's ``lse [T]`` from :func:`more_route_ex` on the same inputs (Algorithm 2)."""
    T, h = X.shape
    r, M = R2.shape
    rc = lib().more_route_psum(_ptr(X), _ptr(R1), _ptr(R2), T, h, r, M, _ptr(lse), _ptr(out_psum), path, _stream(stream))
    if rc != 0:
        raise MoreRouteError(rc, "more_route_psum")


def more_dispatch(idx, counts, out_offsets, out_sorted_pairs, stream=None):
    """``more_dispatch`` of the C interface: from ``idx [T,k]`` and ``counts [M]`` (int32, as written by
    :func:`more_route`) fill ``out_offsets [M+1]`` (exclusive prefix sum of the counts) and ``out_sorted_pairs [T*k]``
    (flat positions ``token*k + slot`` grouped by expert; order inside an expert's run unspecified)."""
    T, k = idx.shape
    M = counts.shape[0]
    rc = lib().more_dispatch(_ptr(idx), _ptr(counts), T, k, M, _ptr(out_offsets), _ptr(out_sorted_pairs), _stream(stream))
    if rc != 0:
        raise MoreRouteError(rc, "more_dispatch")


def more_route_full(X, W, k, gate_mode, out_idx, out_gate, out_counts, out_topval=None, out_lse=None, msplit=0,
                    stream=None):
    """``more_route_full`` of the C interface: the fused standard router, logits ``X [T,h] @ W [h,M]`` (bf16, device)."""
    T, h = X.shape
    M = W.shape[1]
    rc = lib().more_route_full(_ptr(X), _ptr(W), T, h, M, k, gate_mode, _ptr(out_idx), _ptr(out_gate), _ptr(out_counts),
                               _ptr(out_topval), _ptr(out_lse), msplit, _stream(stream))
    if rc != 0:
        raise MoreRouteError(rc, "more_route_full")


def more_merge_shards(idx, topval, lse, shard_base, M, gate_mode, out_idx, out_gate, out_counts, out_topval=None,
                      out_lse=None, stream=None):
    """``more_merge_shards`` of the C interface: ``idx``/``topval`` ``[S,T,k]`` (device), ``lse`` ``[S,T]`` or None,
    ``shard_base`` a host sequence of S ints or None; fills ``out_idx``/``out_gate`` ``[T,k]`` and ``out_counts [M]``."""
    S, T, k = idx.shape
    base = None
    if shard_base is not None:
        base = (ctypes.c_int32 * S)(*[int(b) for b in shard_base])
    rc = lib().more_merge_shards(_ptr(idx), _ptr(topval), _ptr(lse) if lse is not None else None,
                                 ctypes.cast(base, ctypes.c_void_p) if base is not None else None,
                                 S, T, k, M, gate_mode, _ptr(out_idx), _ptr(out_gate),
                                 _ptr(out_topval) if out_topval is not None else None,
                                 _ptr(out_lse) if out_lse is not None else None, _ptr(out_counts), _stream(stream))
    if rc != 0:
        raise MoreRouteError(rc, "more_merge_shards")


def more_route_status(stream=None) -> int:
    return int(lib().more_route_status(_stream(stream)))


def debug_expire_wait(budget_cycles: int, stream=None) -> int:
    """Diagnostic: run the library's bounded mbarrier wait on a barrier nobody arrives at, so that it runs out after
    ``budget_cycles`` clocks and leaves ``MORE_ERR_TIMEOUT`` for :func:`more_route_status` (nothing hangs or faults)."""
    return int(lib().more_debug_expire_wait(budget_cycles, _stream(stream)))


def debug_scratch_guard(stream=None) -> int:
    """Diagnostic: 1 if the guard region behind the library's scratch allocation is intact, 0 if it was written to."""
    return int(lib().more_debug_scratch_guard(_stream(stream)))


@dataclass
class RouteResult:
    idx: "object"
    gate: "object"
    counts: "object"
    topval: "object" = None
    lse: "object" = None


def route(X, R1, R2, k, gate_mode=GATE_TOPK_SOFTMAX, want_topval=False, want_lse=False, path=PATH_AUTO, msplit=0,
          stream=None) -> RouteResult:
    """Convenience wrapper: allocate the outputs with torch and call :func:`more_route_ex`."""
    import torch
    T = X.shape[0]
    M = R2.shape[1]
    dev = X.device
    idx = torch.empty((T, k), dtype=torch.int32, device=dev)
    gate = torch.empty((T, k), dtype=torch.float32, device=dev)
    counts = torch.empty((M,), dtype=torch.int32, device=dev)
    topval = torch.empty((T, k), dtype=torch.float32, device=dev) if want_topval else None
    lse = torch.empty((T,), dtype=torch.float32, device=dev) if want_lse else None
    more_route_ex(X, R1, R2, k, gate_mode, idx, gate, counts, topval, lse, path, msplit, stream)
    return RouteResult(idx, gate, counts, topval, lse)
