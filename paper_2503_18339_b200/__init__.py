"""GranQ channel-wise activation fake-quantization for NVIDIA B200 (sm_100a).

`binding` wraps the C ABI of libgranq.so (include/granq.h); `workloads` holds the seeded
synthetic activation sets; `build` compiles the library in-tree with nvcc.
"""
from . import workloads  # noqa: F401  (pure numpy, importable without the CUDA library)

__all__ = ["binding", "build", "workloads"]
