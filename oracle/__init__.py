"""CPU oracle of the AutoAssist batch-generator hot path (test infrastructure).

Only the tests, the smoke check and the benchmark's CPU-baseline leg import
this package.  It shares nothing with the CUDA library.
"""
