"""CPU oracle for the dense-decoder train step.  TEST INFRASTRUCTURE ONLY.

Nothing on the product path may import this package: only the tests, the
smoke check and the benchmark's CPU-baseline leg do.  It shares no code with
the CUDA library.
"""
