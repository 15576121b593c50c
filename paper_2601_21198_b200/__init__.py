"""B200-native lossless decode of compressed bf16 MoE expert weights (ZipMoE hot path).

`paper_2601_21198_b200.binding` is the thin ctypes layer over the C-ABI
library (include/zipmoe.h); importing it fails loudly when the CUDA library has
not been built.  `paper_2601_21198_b200.inputs` draws the seeded synthetic
tensors and depends on nothing else in the package.
"""
__all__ = ["binding", "inputs", "build"]
