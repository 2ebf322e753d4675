"""Float64 CPU oracle for the DP-SGD hot path.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this; only the
tests, the smoke check and the benchmark's CPU-baseline leg do.  It shares no
code with the CUDA path.
"""
