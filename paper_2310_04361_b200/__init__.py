"""B200-native dynamic-k MoE layer (D2DMoE inference hot path, arXiv 2310.04361).

`paper_2310_04361_b200.api` is the thin binding over the C-ABI CUDA library
(`include/d2d.h`); `paper_2310_04361_b200.workloads` draws the seeded synthetic
inputs.  Importing the package itself loads nothing, so the input generators
stay usable on a machine without the built library; importing `api` fails
loudly when the library is missing.
"""
__all__ = ["api", "workloads", "build"]
