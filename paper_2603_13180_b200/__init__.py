"""B200-native MXNorm hot path: fused per-token normalise-and-quantise kernels behind a C ABI.

``paper_2603_13180_b200.workloads`` holds the seeded input recipes; the binding to the CUDA
library lives in ``paper_2603_13180_b200.binding`` and is imported on first use so that the input
recipes stay importable without the compiled library.
"""
__all__ = ["workloads"]
