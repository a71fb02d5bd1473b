"""B200-native hot path of Multi-Scale Dequant (MSD): hand-written sm_100a kernels behind a C ABI.

``binding`` marshals torch tensors into the C-ABI calls declared in ``include/msd.h``;
``inputs`` holds the seeded synthetic workloads.  There is no CPU fallback: every call fails
loudly when the CUDA library is missing.
"""
__all__ = ["binding", "inputs", "build"]
