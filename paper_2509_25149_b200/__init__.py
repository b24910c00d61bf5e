"""B200-native NVFP4 quantize + block-scaled FP4 GEMM path (sm_100a CUDA behind a C ABI).

``paper_2509_25149_b200.binding`` marshals torch device tensors into the C-ABI calls
declared in ``include/nvfp4.h``; ``paper_2509_25149_b200.synth`` draws the seeded
synthetic inputs.  Importing the package itself loads nothing native.
"""
__all__ = ["binding", "synth", "build"]
