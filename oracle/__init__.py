"""CPU oracle of the sparse-bitmap codec. TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library and its Python binding never do.
"""
