"""fp64 CPU oracle of the global-resolution verification rule.

Test infrastructure only: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg; never by the CUDA package.
"""
