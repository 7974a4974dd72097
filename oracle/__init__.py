"""CPU oracle for the FP4 linear layer (test infrastructure, not a product path).

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
import this package.  The CUDA library never does, and nothing here imports the
CUDA package.
"""
