"""B200-native LAWCAT layer: hand-written sm_100a kernels behind a C ABI, with a thin Python binding.

Importing the package loads nothing; the CUDA library is opened on first use of :mod:`.api`.
"""
__all__ = ["api", "inputs", "build"]
__version__ = "0.1.0"
