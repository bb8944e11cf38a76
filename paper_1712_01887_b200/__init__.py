"""B200-native Deep Gradient Compression hot path (C-ABI CUDA library + thin binding).

`paper_1712_01887_b200.binding` loads the CUDA library (and fails loudly if it
is missing); `paper_1712_01887_b200.inputs` only generates seeded synthetic
gradients and loads nothing.
"""
