"""CPU oracle for the attention path (plain C, IEEE f64).

TEST INFRASTRUCTURE ONLY: the test-suite, the smoke check and the benchmark's
cpu-baseline / reference legs may import this package; the CUDA library and its
Python binding never do, and nothing here imports them.
"""
