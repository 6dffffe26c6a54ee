"""CPU oracle package: test infrastructure only.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import it.
The CUDA library and its Python binding never do.
"""
