"""Triangle-block SYRK for NVIDIA B200: CUDA kernels behind a C ABI (libtbsyrk.so),
with a thin ctypes binding (``binding``) and seeded input generators (``inputs``).

Nothing is imported eagerly: ``inputs`` works without the shared library, while
``binding`` raises if the library has not been built.
"""
