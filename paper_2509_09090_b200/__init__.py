"""B200-native (sm_100a) implementation of the SQAP-VLA hot path: W4A4 linears on a
visual-token set reduced by the paper's quantization-aware pruning criterion.

The product is the C-ABI library built from ``csrc/`` (declared in ``include/sqap.h``);
``binding`` is the thin ctypes layer over it and ``workloads`` the seeded input generators.
Nothing here computes on the CPU: if the CUDA library is missing, calls raise.
"""
__all__ = ["binding", "workloads", "build"]
