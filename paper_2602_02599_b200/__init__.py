"""B200-native RAP decode path: thin Python binding over the C-ABI CUDA library.

Importing the package does not load the library; the first call into the binding does,
and raises if the built shared object is missing (there is no CPU fallback).
"""
