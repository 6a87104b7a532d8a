"""B200-native batched verify-and-resample for Cool-SD (annealed relaxed speculative decoding)."""
