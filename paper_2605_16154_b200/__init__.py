"""B200-native GRPO actor update with Probabilistic Chunk Masking.

`synth` (seeded input generators) imports without the CUDA library; everything in `binding`
needs the compiled shared library and raises if it is missing.
"""
