"""B200-native batched environment stepping (CUDA library + thin ctypes binding).

Importing the package does not load the CUDA library; the first call into
`paper_2207_07736_b200.binding` does, and raises if the library has not been built.
"""
__all__ = ["inputs", "binding", "build"]
