"""B200-native GaLore-Adam optimizer step (arXiv 2403.03507, Algorithm 1).

The compute lives in a C-ABI CUDA library (`include/galore.h`); `binding`
marshals arguments to it.  Importing the package does not load the library:
`paper_2403_03507_b200.binding` does, and raises if it is missing.
"""
