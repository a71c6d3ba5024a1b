"""CPU oracle for the GEMM hot path -- TEST INFRASTRUCTURE, not part of the product.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
It shares no code with the CUDA library; neither imports the other.
"""
