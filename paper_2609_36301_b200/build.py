"""Build ``libmore_route.so`` in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_HERE, "csrc")
LIB_PATH = os.path.join(_HERE, "libmore_route.so")
SOURCES = ["more_route_api.cu", "more_route_generic.cu", "more_route_sm100.cu", "more_route_full_sm100.cu",
           "more_route_noalloc.cu",
           "more_dispatch.cu", "more_psum_sm100.cu", "more_merge.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC"]


def _newest_source_mtime() -> float:
    paths = [os.path.join(_CSRC, f) for f in os.listdir(_CSRC)]
    paths.append(os.path.join(os.path.dirname(_HERE), "include", "more_route.h"))
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False, out: str | None = None, defines: tuple = ()) -> str:
    """Compile the CUDA sources if the library is missing or older than any source; return its path.

    ``defines`` adds ``-D`` switches (the diagnostic builds: ``MORE_STATS`` for event and clock counters,
    ``MORE_EXP_NOSCAN`` / ``MORE_EXP_NOPROC`` / ``MORE_EXP_NOFOLD`` for the epilogue with its candidate handling,
    everything but the tensor-memory loads, or its folds compiled out; ``MORE_DEV`` for the ``MORE_KERNEL=p|g`` and
    ``MORE_PLAN=block_tokens,es,msplit,filter`` environment overrides of the launch plan; ``MORE_PAIRED_DBL=0`` for the
    paired kernel with z in tensor memory at every rank; ``MORE_WITH_FILTER`` for the experimental filter sweep;
    ``MORE_CAND_CAP=n`` candidate slots per token); such a build goes to ``out``, never over the product library."""
    target = out or LIB_PATH
    if defines and target == LIB_PATH:
        raise ValueError("a diagnostic build needs its own output path")
    if not force and os.path.exists(target) and os.path.getmtime(target) >= _newest_source_mtime():
        return target
    nvcc = os.environ.get("NVCC", "nvcc")
    cmd = [nvcc] + NVCC_FLAGS + ["-D" + d for d in defines] + (["-Xptxas", "-v"] if verbose else []) + \
          ["-o", target] + [os.path.join(_CSRC, s) for s in SOURCES]
    subprocess.run(cmd, check=True)
    return target


if __name__ == "__main__":
    import sys
    # python -m paper_2609_36301_b200.build [OUT.so DEFINE ...]
    if len(sys.argv) > 2:
        print(build(force=True, out=sys.argv[1], defines=tuple(sys.argv[2:])))
    else:
        print(build(force=True, verbose=True))
