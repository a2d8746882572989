"""CPU float64 oracle for the Mutual-RL token-level policy-loss pass.

TEST INFRASTRUCTURE ONLY.  Nothing here is part of the product: only the
tests, the smoke check and the benchmark's CPU-baseline leg may import it.
It shares no code with the CUDA path and never imports the package.
"""
