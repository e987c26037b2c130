"""B200-native dense BLAS level-1 / level-2 kernel family behind a C-ABI library.

``binding`` holds the ctypes front-end of ``libb2blas.so`` (hand-written sm_100a CUDA);
``synth`` holds the seeded input generators; ``build`` compiles the library in-tree.
Nothing here falls back to a CPU implementation: without the compiled CUDA library every
routine raises.
"""

__all__ = ["binding", "synth", "build"]
