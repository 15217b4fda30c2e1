"""AG-gated attention layer for B200: CUDA library + thin ctypes binding.

Importing the package does not load the CUDA library; `binding` does, on
first use, and raises if the library has not been built.
"""
