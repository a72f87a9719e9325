"""fp64 CPU oracle for the ReHyAt hybrid attention operator.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this package;
only the tests, the smoke check and the bench's CPU-baseline leg do.  It shares
no code with the CUDA path.
"""
