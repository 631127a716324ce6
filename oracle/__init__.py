"""TEST INFRASTRUCTURE ONLY: the plain CPU statement of the routing simulator.

Only tests, the smoke check and the timed CPU-baseline leg of the benchmark may import
this package; the CUDA library and its Python binding never do.
"""
