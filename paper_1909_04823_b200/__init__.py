"""B200-native hot path of Distributed Equivalent Substitution training
(arXiv 1909.04823): a C-ABI CUDA library (`libdes.so`, declared in
include/des.h) and a thin ctypes binding.

`synth` (numpy-only input generators) imports nothing else of the package;
`binding` loads the CUDA library and fails loudly when it cannot."""
__all__ = ["synth", "binding", "build"]
