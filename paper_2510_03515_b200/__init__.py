"""B200-native importance-weighted group-advantage policy-gradient loss (RAPID, arXiv 2510.03515).

The product is the CUDA library behind the C ABI declared in include/rapid_pg.h; `binding` is a
thin ctypes layer over it (argument marshalling only) and `synth` draws the seeded synthetic
inputs.  Importing the package does not load the library; the first call through `binding`
does, and raises if the library has not been built.
"""

__all__ = ["binding", "synth", "build"]
