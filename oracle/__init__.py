"""Slow, plain CPU references for the SYRK path (test infrastructure only).

``oracle.syrk`` - the numeric definition (Algorithm 1 plus alpha/beta), in C.
``oracle.tbs``  - the triangle-block schedule and its I/O count, in integers.

Nothing here is imported by the GPU library or its Python binding.
"""
