"""CPU oracle for the action-conditioned decode step (test infrastructure).

Nothing in the product package imports this directory.  Only the tests, the
smoke check and the benchmark's CPU-baseline leg may call it.
"""
