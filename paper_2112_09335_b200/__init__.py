"""Community-based ADMM training of graph convolutional networks on one B200.

The package holds the Python binding of the C-ABI library (``binding``), the CUDA
sources it is built from (``csrc/``) and the seeded synthetic input generators
(``inputs``).  Importing the package loads nothing heavy; ``binding`` loads the
shared library on first use and raises if it has not been built.
"""

__all__ = ["inputs", "binding", "build"]
