"""B200-native multiquery decode attention over a KV cache (sm_100a)."""
