"""fp64 CPU oracle for the ADMM-Q layer solver.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this package:
only the tests, the smoke check and the benchmark's CPU-baseline / reference
arm call it.  It shares no code with the CUDA path.
"""
