"""B200-native batched what-if timing/energy evaluation over kernel dependency graphs.

`paper_2607_12324_b200.emo` is the thin Python binding over the C-ABI library (loaded on first
use; it raises if the CUDA library has not been built).  `paper_2607_12324_b200.workloads` holds
the seeded synthetic input generators and imports nothing from the CUDA path.
"""
__all__ = ["workloads"]
