"""CPU oracle (test infrastructure only): the plain definition the CUDA library is checked against.

Only tests, the smoke check and the benchmark's cpu_baseline / reference legs import this package.
"""
