"""B200-native decode-step attention of TidalDecode's position persistent sparse
attention: a C-ABI CUDA library (csrc/, include/tidal.h) and its ctypes binding.

Nothing is imported eagerly: `binding` loads (and if needed builds) libtidal.so,
`synth` makes the seeded synthetic inputs used by tests and benchmarks."""

__all__ = ["binding", "build", "synth"]
