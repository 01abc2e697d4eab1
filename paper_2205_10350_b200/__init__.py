"""B200-native verification step of Aggressive Decoding (arXiv 2205.10350).

``binding`` wraps the C ABI of ``libad_b200.so`` (hand-written sm_100a kernels); ``synth`` draws the seeded
synthetic inputs; ``build`` compiles the library in-tree.  Nothing is imported eagerly so that the input
generator can be used on machines without CUDA.
"""
