"""B200-native HBF service model: the batch hot path of HBFSim's method as CUDA kernels behind a
C-ABI library (``libhbf.so``), with a thin ctypes binding.

``workloads`` (seeded synthetic inputs) imports without a GPU.  The binding (``hbf``) loads the
CUDA library on first use and raises if it has not been built; there is no CPU fallback.
"""
__all__ = ["workloads", "hbf"]
