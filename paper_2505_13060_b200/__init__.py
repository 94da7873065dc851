"""B200-native loss-MSE sensitivity pass (automatic mixed precision, Algorithm 1 steps 2 and 4).

``binding`` is the thin ctypes layer over the C-ABI library (``include/ampq.h``);
``synth`` holds the seeded synthetic input recipes and none of the method's
arithmetic.  Importing the package does not load the CUDA library; the first
use of ``binding`` does, and fails loudly if it has not been built.
"""
