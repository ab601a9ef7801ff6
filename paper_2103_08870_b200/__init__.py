"""B200-native implementation of the Learned Gradient Compression (LGC) per-step path.

``workloads`` makes seeded synthetic inputs; ``lgc`` is the thin binding of the C-ABI CUDA
library (loaded on first use; importing this package needs neither a GPU nor the built library).
"""
__all__ = ["workloads", "lgc", "build"]
