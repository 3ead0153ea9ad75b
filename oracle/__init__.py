"""Independent CPU checker for decode attention (test infrastructure, not product code).

Only tests, the smoke check and the benchmark's CPU-baseline leg import this package; the
CUDA library and its Python binding never do, and nothing here imports them.
"""
