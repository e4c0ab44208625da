"""B200-native LTE sparse-attention hot path (scores, select, prefill, decode, backward).

``paper_2510_20787_b200.lte`` is the thin binding over the C-ABI CUDA library;
``paper_2510_20787_b200.synth`` is the seeded input generator (no method arithmetic).
Nothing is imported eagerly so that the generator can be used without the library.
"""
