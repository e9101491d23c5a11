"""B200-native BP-Transformer graph self-attention (arXiv 1911.04070)."""
