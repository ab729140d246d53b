"""DS-FACTO training hot path (doubly-separable factorization-machine epoch) for NVIDIA B200.

`paper_2004_13940_b200.dsfacto` is the ctypes binding of the CUDA C-ABI library declared in
include/dsfacto.h; `paper_2004_13940_b200.workloads` produces the seeded synthetic inputs.
Nothing here falls back to the CPU: the binding raises if the CUDA library is missing."""

__all__ = ["dsfacto", "workloads", "build"]
