"""B200-native pool attention: causal, sample-masked attention forward and backward
over a pool of packed sequences, scheduled as weighted SH-Tiles on persistent CTAs.

Importing the package is cheap and touches no GPU.  `paper_2607_23250_b200.binding`
loads the CUDA library (and raises if it has not been built); `pools` holds the
seeded input generators.
"""
__all__ = ["pools", "binding", "build"]
