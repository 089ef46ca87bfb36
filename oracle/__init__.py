"""CPU oracle for the LoPRo quantized-linear forward.

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain, fp64 statement of
what the method computes, written from the paper's equations.  It shares no
code with the CUDA library and is never imported by it.  Only the tests, the
smoke check and the CPU-baseline leg of the benchmark may use it.
"""
