"""B200-native HiSpec verification path (hierarchical speculative decoding on an
early-exit transformer): a C-ABI CUDA library plus a thin Python binding.

Importing the package does not load the CUDA library; `binding.load()` does,
and raises if the library has not been built."""
__all__ = ["workload", "binding", "driver", "build"]
