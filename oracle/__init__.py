"""CPU oracle (test infrastructure): the plain definition of what the CSB-RNN
hot path computes.  Only tests, the smoke check and the benchmark's CPU-baseline
leg may import this package; the CUDA library never does."""
