"""CPU oracle of the MoE expert step: test infrastructure only.

Only tests, the smoke check and the benchmark's cpu_baseline leg import this package; the
product path never does.
"""
