"""B200-native ADORE decode path: thin Python binding over the C ABI in include/adore.h.

Importing the package does not load the CUDA library; `paper_2407_02328_b200.adore` does,
and fails loudly if it has not been built (`python -m paper_2407_02328_b200.build`).
"""
__all__ = ["adore", "build"]
