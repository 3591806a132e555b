"""Head-local weighted affine ridge mapping of KV caches on B200: CUDA library + thin binding.

`synth` holds the seeded input generators; `binding` mirrors the C ABI of include/cb.h; `build` compiles the
library in-tree.  Nothing here computes on the CPU.
"""
