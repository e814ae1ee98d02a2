"""CPU oracle for the structured contraction ops: test infrastructure only.

Nothing in the product path imports this package; only tests, the smoke check
and the benchmark's CPU-baseline leg do.
"""
