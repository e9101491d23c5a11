"""B200-native BP-Transformer graph self-attention (arXiv 1911.04070).

``binding`` wraps the C ABI of libbpt.so; ``synth`` draws seeded inputs;
``build`` compiles the CUDA sources.
"""
