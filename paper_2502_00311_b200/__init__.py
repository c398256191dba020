"""B200-native CUDA implementation of the per-step hot path of Sparse Gradient Compression.

`paper_2502_00311_b200.binding` wraps the C-ABI library (include/sgc.h); it is loaded lazily and
raises if the compiled library is missing.  `paper_2502_00311_b200.inputs` holds the seeded
synthetic input generators.
"""
__all__ = ["binding", "inputs", "build"]
