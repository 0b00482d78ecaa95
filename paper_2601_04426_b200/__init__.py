"""B200-native token-mask hot path for grammar-constrained decoding (byte-level Earley).

`paper_2601_04426_b200.binding` is the thin ctypes layer over the C-ABI library (libxg.so, built
in-tree from csrc/ by `paper_2601_04426_b200.build`).  `paper_2601_04426_b200.inputs` holds the
seeded synthetic input generators.  Nothing is imported eagerly: importing the package never loads
the CUDA library.
"""
__all__ = ["binding", "build", "inputs"]
