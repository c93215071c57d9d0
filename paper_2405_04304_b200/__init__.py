"""B200-native logit tails of DISCO speculative decoding (arXiv 2405.04304).

``paper_2405_04304_b200.binding`` wraps the C-ABI CUDA library (libdisco.so);
``paper_2405_04304_b200.inputs`` draws the seeded synthetic inputs.  Importing
the package itself loads nothing; the binding loads the library on first use and
raises if it has not been built.
"""

__all__ = ["binding", "inputs"]
