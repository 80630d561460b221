"""TEST INFRASTRUCTURE -- the CPU oracle and simulators.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  Nothing under ``paper_2509_25224_b200`` does.
"""
