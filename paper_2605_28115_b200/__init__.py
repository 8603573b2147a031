"""B200-native select + compact + KV-compaction path of CIVIC (sm_100a CUDA, C-ABI)."""
