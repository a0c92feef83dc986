"""B200-native TSP gated ring MLP (Algorithm 2): C-ABI CUDA library plus a thin binding.

Importing the package does not load the CUDA library; the first call into
:mod:`paper_2604_26294_b200.binding` does, and fails loudly if it is missing.
"""
