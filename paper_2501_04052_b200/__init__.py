"""B200-native RaZeR matmul path (arXiv 2501.04052): CUDA kernels behind a C ABI.

`binding` loads the compiled library and exposes the C entry points one to one;
`inputs` draws the seeded synthetic tensors.  Importing the package does not load
the library; importing `binding` does, and fails loudly if it has not been built.
"""
__all__ = ["binding", "inputs", "build"]
