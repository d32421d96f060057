"""B200-native draft-tree verification (speculative-decoding verify step)."""
