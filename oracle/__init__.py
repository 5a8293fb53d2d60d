"""CPU oracle of the MXFP4 backward pass: TEST INFRASTRUCTURE ONLY.

Only the test-suite, the smoke check and the CPU-baseline leg of the benchmark
may import this package.  The CUDA library never does, and shares no code with
it.  ``oracle.ref`` is a ctypes view of ``mxfp4_oracle.c``.
"""
