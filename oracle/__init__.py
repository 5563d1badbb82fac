"""CPU oracle of the constrained-MMSE quantization path (test infrastructure only).

Nothing in the CUDA library imports this package; it exists so that the tests, the smoke
check and the benchmark's CPU-baseline leg have an independent statement of the method.
"""
