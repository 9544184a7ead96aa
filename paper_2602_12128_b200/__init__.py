"""B200-native Hadamard Linear Attention operator (linear-time HLA, forward and
backward) behind a C-ABI CUDA library.  Importing the package loads nothing
heavy; the shared library is loaded on first use of `binding`."""
__all__ = ["synth", "flops", "binding", "build"]
