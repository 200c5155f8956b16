"""B200-native (sm_100a) multiquery decode attention over a KV cache.

``binding`` wraps the C ABI of ``include/mqa_decode.h``; ``build`` compiles the
CUDA sources in-tree; ``roofline`` holds the byte/flop accounting.
"""
