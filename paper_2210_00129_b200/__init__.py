"""B200-native Stochastic Backpropagation (SBP) linear-layer hot path.

The compute lives in a C-ABI CUDA library (``include/sbp.h``); this package is
its thin Python binding plus the seeded input generators (``synth``).
"""
