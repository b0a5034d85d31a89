"""CPU oracle of the ReFreeKV post-prefill compression pass (test infrastructure).

Only the tests, the smoke check and the benchmark's CPU-baseline leg import
this package; the CUDA product path never does.
"""
