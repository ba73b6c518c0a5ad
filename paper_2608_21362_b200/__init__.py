"""kvb: B200-native KV-chunk stitching (dequantise, re-rotate, scatter), cosine-deviation
top-k selection and selective causal attention.  The CUDA library is loaded on first use by
``paper_2608_21362_b200.binding``; there is no CPU fallback."""
