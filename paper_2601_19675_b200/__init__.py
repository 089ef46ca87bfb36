"""B200-native forward of a LoPRo-quantized linear layer (C-ABI library + thin binding).

`paper_2601_19675_b200.lopro` is the ctypes binding of the CUDA library (loaded on first
use; it raises if the library has not been built).  `paper_2601_19675_b200.synth` holds
the seeded synthetic input generators.
"""
__all__ = ["lopro", "synth"]
