"""B200-native MDBF quantized linear forward (libmdbf) — Python binding.

`paper_2512_24545_b200.mdbf` wraps the C-ABI shared library one-to-one;
`paper_2512_24545_b200.inputs` holds the seeded synthetic input generators.
Importing the package does not load the CUDA library; the first call into
`mdbf` does, and fails loudly when the library has not been built.
"""
__all__ = ["inputs", "mdbf"]
