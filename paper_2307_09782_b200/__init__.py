"""B200-native W4A8 quantized linear layer (FP4-E2M1 weights, FP8-E4M3 activations, LoRC).

``synth`` draws the seeded synthetic inputs; ``binding`` is the thin ctypes layer over the C-ABI
library built from ``csrc/``.  Importing the package does not load the CUDA library.
"""
