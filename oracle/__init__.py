"""TEST INFRASTRUCTURE: the CPU oracle.

A plain, slow, scalar implementation of the vocabulary index (Algorithms 3 and
4 of the paper) and of the masked greedy decode step (Algorithm 2), used to
check the CUDA library.  It shares no code with that library and neither
imports the other.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may use this package; the product never does.
"""
