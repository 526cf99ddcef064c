"""B200-native quantized-pruning KV-cache hot path (arXiv 2412.12706).

``paper_2412_12706_b200.qp`` is the thin binding over the C-ABI CUDA library;
``paper_2412_12706_b200.synth`` produces the seeded synthetic inputs.  Nothing
here falls back to a CPU implementation: calling into ``qp`` without the built
CUDA library raises.
"""
