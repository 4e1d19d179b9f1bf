"""B200 (sm_100a) C-step of the learning-compression scheme: CUDA kernels behind
a C ABI (``include/condensa_cstep.h``) and a thin ctypes binding (``cstep``).
``workloads`` holds the seeded synthetic weight sets."""
__all__ = ["cstep", "workloads", "build"]
