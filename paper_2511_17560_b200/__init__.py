"""B200-native hot path of attention-aware KV-cache fusion (A^3).

`paper_2511_17560_b200.a3` is the thin binding over the C-ABI library (liba3.so); it
raises at first use when the CUDA library has not been built.  `workloads` holds the
seeded synthetic input generators.
"""
