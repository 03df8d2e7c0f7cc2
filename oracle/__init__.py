"""CPU oracle for the AdaComp pack / unpack-sum path.  TEST INFRASTRUCTURE ONLY.

Nothing in the product package may import this; only the tests, the smoke
check and the benchmark's CPU-baseline leg do.  It shares no code with the
CUDA library.
"""
