"""B200-native verification hot path of speculative decoding with Cross-model Retrieval."""
