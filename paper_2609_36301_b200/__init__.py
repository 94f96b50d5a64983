"""B200-native fused low-rank MoE router (MoRE): ctypes binding over hand-written sm_100a CUDA kernels.

``from paper_2609_36301_b200 import binding`` gives the C interface (see ``include/more_route.h``);
``inputs`` holds the seeded synthetic workloads used by the tests and the benchmark.
"""
__all__ = ["binding", "inputs", "build"]
