"""B200-native "stairs" assisted greedy generation: the large model's validation pass.

`workloads` (pure data generators) can be imported without the CUDA library;
`stairs` (the binding over the C-ABI shared library) fails loudly if the library
has not been built.
"""
