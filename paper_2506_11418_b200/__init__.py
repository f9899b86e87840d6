"""B200-native CentroidKV hot path: Chunked Soft Matching KV-cache clustering and
decode attention over the compressed cache, behind a C-ABI library (see include/ckv.h).

The CUDA library is loaded on first use of `paper_2506_11418_b200.binding`; nothing here
falls back to a CPU implementation.
"""
__all__ = ["binding", "synth", "build"]
