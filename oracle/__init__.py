"""CPU fp64 oracle for the RMM linear layer: test infrastructure only.

Nothing in the product package imports this; only the tests, the smoke check
and the benchmark's CPU-baseline leg do.
"""
