"""B200-native hot path of Mosaic's composite projection pruning.

`paper_2504_06323_b200.api` is the thin binding over the C-ABI CUDA library
(`libmosaic.so`, built from `csrc/`); `workloads` generates the seeded
synthetic inputs; `driver` runs the path over a whole LLaMA-shaped model.
"""
__all__ = ["api", "workloads", "driver"]
