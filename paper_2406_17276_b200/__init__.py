"""B200-native OPT-Tree draft-tree construction, tree mask and greedy verification.

`binding` wraps the C ABI of the CUDA library (include/opt_tree.h); `synth` holds the
seeded input generators; `build` compiles the library in-tree.
"""
