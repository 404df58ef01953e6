"""CPU oracle for SuffixDecoding draft generation: test infrastructure only.

`SuffixOracle` wraps the plain C++ implementation in ``suffix_oracle.cpp``
(built with g++ by :func:`build`).  Nothing under this package may be imported
by the CUDA library or its Python binding.
"""
from .binding import SuffixOracle, build, library_path  # noqa: F401
