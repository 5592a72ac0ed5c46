"""CPU oracle for the GG pass: test infrastructure only.

Only the tests, the smoke check and the benchmark's CPU-baseline leg import
this package; the CUDA library and its Python binding never do.
"""
