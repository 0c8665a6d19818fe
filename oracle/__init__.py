"""CPU checker ("oracle") for the verification round and the bandit updates.

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
CPU-baseline leg of the benchmark.  The product path never imports it, and it
imports nothing from the product.
"""
