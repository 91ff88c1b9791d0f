"""TEST INFRASTRUCTURE: the CPU oracle.  Only tests, the smoke check and the CPU-baseline
leg of the bench may import this package; the product path never does."""
