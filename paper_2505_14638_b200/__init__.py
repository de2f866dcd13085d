"""B200-native W4A8 linear layer (INT4-stored weights, FP8 E4M3 math) after Sec. 3 of
"Dual Precision Quantization": hand-written sm_100a kernels behind a C-ABI library, with a thin
ctypes binding.  Importing the package does not load the CUDA library; the first call does, and
fails loudly when it has not been built."""

__all__ = ["binding", "inputs", "build"]
