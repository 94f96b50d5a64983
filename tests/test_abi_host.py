"""Host-side checks that need no GPU: the shared library loads, exports every symbol the header declares,
rejects bad arguments before touching a device, and plans launches sensibly."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2609_36301_b200 import binding as mr
from paper_2609_36301_b200 import build as mr_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "more_route.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(more_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    mr_build.build()
    lib = mr.lib()
    names = declared_functions()
    assert {"more_route", "more_route_ex", "more_route_host", "more_route_plan", "more_route_status",
            "more_strerror", "more_version", "more_route_launches"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in more_route.h but not exported"
    assert mr.version() >= 100
    assert "ok" == mr.strerror(0)


def test_bad_arguments_are_rejected_before_any_device_work():
    lib = mr.lib()
    buf = (ctypes.c_char * 4096)()
    p = ctypes.addressof(buf)
    p16 = (p + 15) & ~15
    def call(X=p16, R1=p16, R2=p16, T=4, h=8, r=8, M=8, k=2, mode=0, idx=p16, gate=p16, counts=p16):
        return lib.more_route(X, R1, R2, T, h, r, M, k, mode, idx, gate, counts, None)
    assert call(k=9) == -2            # k > M
    assert call(k=0) == -2
    assert call(T=-1) == -2
    assert call(M=40, k=33) == -2     # k > MORE_K_MAX
    assert call(r=2048) == -2         # r > MORE_R_MAX
    assert call(M=(1 << 30) + 8) == -2   # M > MORE_M_MAX
    assert call(mode=2) == -4
    assert call(X=None) == -1
    assert call(counts=None) == -1
    assert call(X=p16 + 2) == -3
    assert call(idx=p16 + 1) == -3
    assert lib.more_route_ex(p16, p16, p16, 4, 8, 8, 8, 2, 0, p16, p16, p16, None, None, 7, 0, None) == -4
    for code in range(-8, 1):
        assert len(mr.strerror(code)) > 1


def test_plan_picks_paths_and_splits():
    P = mr.more_route_plan
    assert P(256, 128, 8, 256, 2).path == mr.PATH_TCGEN05
    assert P(100, 20, 5, 33, 3).path == mr.PATH_GENERIC          # odd sizes
    assert P(64, 64, 96, 256, 4).path == mr.PATH_GENERIC         # r > 64
    assert P(64, 64, 8, 260, 4).path == mr.PATH_GENERIC          # M % 8 != 0
    with pytest.raises(mr.MoreRouteError):
        P(100, 20, 5, 33, 3, path=mr.PATH_TCGEN05)
    with pytest.raises(mr.MoreRouteError):
        P(300, 256, 32, 4096, 8, msplit=65)                      # more than 64 CTAs per token block
    PX = mr.more_route_plan_ex
    # few token blocks, many experts: the experts are split, inside a CTA and over CTAs, and one wave is not exceeded
    p = PX(8192, 4096, 64, 131072, 16, gate_mode=1)
    assert p.ctas % p.msplit == 0 and p.ctas <= 148
    assert p.msplit * p.expert_ranges >= 4 and p.token_groups * p.expert_ranges <= 4
    # many tokens: the kernel with 256-token CTAs, two per SM, in one wave
    p = PX(65536, 2048, 64, 16384, 8)
    assert p.ctas in range(256, 297) and p.msplit == 1
    # a decode-sized batch is spread over the SMs along the expert axis
    p = PX(64, 2048, 64, 16384, 8)
    assert p.ctas > 16 and p.ctas <= 148 and p.msplit > 1
    # never more CTAs per token block than 64-expert blocks
    assert PX(300, 256, 32, 256, 8, msplit=5).msplit * PX(300, 256, 32, 256, 8, msplit=5).expert_ranges <= 4
    assert P(300, 256, 32, 4096, 8, msplit=5).msplit == 5
    # asking for the log-sum-exp changes the kernel variant but is always accepted
    assert PX(32768, 512, 32, 16384, 8, want_lse=True).path == mr.PATH_TCGEN05


def test_shared_memory_plan_of_the_grouped_kernel_fits():
    """Every (rank, token groups, expert ranges) the planner may pick leaves room for at least two R2 stages and one
    phase-1 stage in the 208 KB ring (checked through the plans of shapes that exercise them)."""
    PX = mr.more_route_plan_ex
    for T in (1, 33, 128, 200, 300, 512, 5000, 20000):
        for r in (8, 16, 32, 64):
            for M in (8, 64, 256, 1000, 4096, 65536):
                for k in (1, 8, 16, 32):
                    if k > M:
                        continue
                    p = PX(T, 512, r, M - M % 8 if M >= 8 else 8, k)
                    assert p.path == mr.PATH_TCGEN05 and p.ctas >= 1
                    assert p.block_tokens % 32 == 0 and 32 <= p.block_tokens <= 512
