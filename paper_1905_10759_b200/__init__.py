"""B200-native Hadamard Binary Matrix Multiply (HadaNets inference path).

``paper_1905_10759_b200.hbmm`` is the binding of the C-ABI library (it loads the
CUDA shared library and fails loudly when it is missing); ``inputs`` holds the
seeded synthetic input generators.  Nothing is imported eagerly here so that the
input generators stay usable without the library.
"""
__all__ = ["hbmm", "inputs"]
