"""CPU oracle for the Q8BERT 8-bit inference path.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package;
the CUDA library and its Python binding never do.
"""
