"""Asymmetry-aware persistent BF16 GEMM for B200 (sm_100a): Python face of the C-ABI library.

``from paper_2609_24270_b200 import binding`` loads the CUDA library (and fails loudly if
it has not been built); ``inputs`` only manufactures seeded synthetic inputs.
"""
