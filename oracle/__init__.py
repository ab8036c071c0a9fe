"""CPU oracle for the PM-KVQ decode hot path.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this
directory; only the test-suite, the smoke check and the benchmark's CPU
baseline leg do.  It shares no code, tables or helpers with the CUDA path.
"""
